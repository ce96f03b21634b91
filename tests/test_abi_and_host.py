"""CPU-only checks: the shared library builds, loads and exports every declared symbol; the workload
generator is deterministic and shaped as documented; host-side argument checks that need no GPU."""
import ctypes
import os
import re

import numpy as np
import torch

from paper_2605_26646_b200 import binding as ub
from paper_2605_26646_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "unity.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(unity_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ub.load_library()
    names = declared_symbols()
    assert set(ub.EXPORTS) <= set(names)
    for n in names:
        assert isinstance(getattr(lib, n), ctypes._CFuncPtr), n


def test_workspace_queries_and_null_context_need_no_gpu():
    lib = ub.load_library()
    full = ub.unity_workspace_bytes(1_600_000, 3584, 152064, 2, 2574)
    least = ub.unity_workspace_min_bytes(1_600_000, 3584, 152064, 2, 2574)
    assert 0 < least < full < 60 * 2 ** 30
    hint = ub.unity_workspace_hint(1_600_000, 3584, 152064, 2)
    assert hint == ub.unity_workspace_bytes(1_600_000, 3584, 152064, 2, 1_600_000) and full <= hint < full + 2 ** 27
    assert ub.unity_workspace_hint(-1, 3584, 152064, 2) == 0
    assert ub.unity_workspace_bytes(-1, 3584, 152064, 2, 1) == 0
    assert lib.unity_check_status(None) == -1
    assert lib.unity_destroy(None) == -1
    assert lib.unity_launch_count(None) == 0
    assert lib.unity_last_error(None) == b"null context"
    assert lib.unity_logprob_fwd(None, None, None, None, None) == -1


def test_generator_is_stateless_and_deterministic():
    a = wl.normal(7, 3, 1000)
    b = torch.cat([wl.normal(7, 3, 400), wl.normal(7, 3, 600, offset=400)])
    assert torch.equal(a, b)
    assert not torch.equal(a, wl.normal(8, 3, 1000)) and not torch.equal(a, wl.normal(7, 4, 1000))
    x = wl.normal(1, 1, 200000).double()
    assert abs(x.mean()) < 0.01 and abs(x.std() - 1) < 0.01
    u = wl.uniform(1, 2, 200000)
    assert 0 < u.min() and u.max() < 1 and abs(u.mean() - 0.5) < 0.005
    r = wl.randint(1, 3, 100000, 5, 9)
    assert r.min() == 5 and r.max() == 8
    w1, w2 = wl.make("tiny"), wl.make("tiny")
    assert torch.equal(w1.hidden, w2.hidden) and torch.equal(w1.W[0], w2.W[0]) and torch.equal(w1.target, w2.target)


def test_configuration_shapes():
    expect = {"tiny": (256, 4096, 1, 2, 64, 1024), "rag_qa": (896, 151936, 1, 2, 1024, None),
              "search": (1536, 151936, 2, 3, None, None), "code": (3584, 152064, 2, 2, None, None),
              "stress": (5120, 152064, 4, 4, 8192, 131072)}
    for name, (H, V, K, R, S, N) in expect.items():
        w = wl.make_structure(name)
        assert (w.H, w.V, w.K, w.n_roles) == (H, V, K, R)
        assert S is None or w.n_inv == S
        assert N is None or w.n_tok == N
        assert int(w.cu_seqlens[-1]) == w.n_tok and w.tok_mask.numel() == w.n_tok
        assert int(w.target.min()) >= 0 and int(w.target.max()) < V
        if name != "code":
            assert 0.75 < w.n_valid / w.n_tok < 0.85
    code = wl.make_structure("code")
    lens = (code.cu_seqlens[1:] - code.cu_seqlens[:-1])
    assert torch.all(lens % 128 == 0) and 1_000_000 < code.n_valid < 1_400_000
    # verifier-score deltas telescope: rewards of a trajectory's coder invocations sum to its last score in [0, 1]
    tot = torch.zeros(code.n_traj, dtype=torch.float64).index_add_(
        0, code.inv_traj.long()[code.inv_role == 0], code.r_turn.double()[code.inv_role == 0])
    assert tot.min() >= -1e-6 and tot.max() <= 1 + 1e-6
    stress = wl.make_structure("stress")
    seg = (stress.inv_group.long() * stress.n_roles + stress.inv_role.long()).numpy()
    r = stress.r_node.numpy()
    seg_std = np.array([r[seg == q].std() for q in range(stress.n_groups * stress.n_roles)])
    assert 0.05 < (seg_std == 0).mean() < 0.16


def test_parity_cut_keeps_structure_and_every_model():
    w = wl.make_structure("stress", cut_rows=300, cut_max_len=64)
    full = wl.make_structure("stress")
    assert w.n_inv == full.n_inv and torch.equal(w.r_node, full.r_node)
    tok_inv = torch.repeat_interleave(torch.arange(w.n_inv), w.cu_seqlens[1:] - w.cu_seqlens[:-1])
    models = w.role_model[w.inv_role.long()[tok_inv]]
    assert set(models.tolist()) == {0, 1, 2, 3} and w.n_tok < 1000
