"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

The fp64 oracle cannot sweep 1.2 M rows x 152 k vocabulary, so the full-size run is checked by
(i) sampled rows the oracle evaluates one by one (log-prob, entropy, token loss and the dHidden row: a row's
    gradient needs only that row, W_k and the global count M_k, so the sampled values are exact at full size),
(ii) the loss against the fp64 sum of the exported per-token losses,
(iii) dW through properties that hold at any size: its column sums over the vocabulary vanish, and it is additive
    over row chunks; one chunk of about a thousand rows per model is checked in full by the oracle (whole tensor
    and per block of 256 vocabulary rows), together with the dHidden rows of the chunk, row by row."""
import numpy as np
import pytest
import torch

import parity_harness as pu
from oracle import unity_oracle as orc
from paper_2605_26646_b200 import binding as ub
from paper_2605_26646_b200 import workloads as wl

pytestmark = pytest.mark.gpu


class DeviceRows:
    """Hands the oracle bf16 bit patterns of the hidden rows it asks for, fetched from the GPU tensor on demand."""

    def __init__(self, t):
        self.t = t
        self.shape = tuple(t.shape)

    def __getitem__(self, idx):
        return pu.bf16_bits(self.t[torch.as_tensor(np.asarray(idx), device=self.t.device)])


@pytest.mark.parametrize("name,n_sample,chunk_rows,stash", [("rag_qa", 192, 1200, False), ("search", 96, 1000, False),
                                                            ("code", 96, 1000, False), ("stress", 64, 600, False),
                                                            ("rag_qa", 192, 1200, True), ("stress", 64, 600, True)])
def test_full_size_sampled_parity(name, n_sample, chunk_rows, stash):
    w = wl.make(name, device="cuda")
    d = pu.DeviceInputs(w)
    ctx = pu.make_ctx(w, stash=stash)
    if stash:          # logit stash instead of the recompute GEMM: several row blocks per model at these sizes
        ctx.set_option(ub.OPT_LOGIT_STASH, 1)
    K, n = w.K, w.n_tok
    role_model = w.role_model.tolist()
    mask_np = w.tok_mask.numpy() != 0
    _, tok_model = orc.token_role_model(w.cu_seqlens.numpy(), w.inv_role.numpy(), w.role_model.numpy())

    # stage 1 at full size against the oracle (cheap)
    ga, oa = pu.gpu_advantage(ctx, w, d), pu.oracle_advantage(w)
    assert np.abs(ga["adv_tok"].cpu().numpy() - oa["adv_tok"]).max() <= pu.TOL_ADV
    adv = ga["adv_tok"]

    # stage 2 gives the current log-probs; old / ref = current + N(0, 0.05) as in the benchmark
    gl = pu.gpu_logprob(ctx, w, d)
    old = gl["logp"] + w.noise_old.cuda()
    ref = gl["logp"] + w.noise_ref.cuda()
    gp = pu.gpu_ppo(ctx, w, d, old, ref, adv)

    # ---- (i) sampled rows, every model represented
    rng = np.random.default_rng(7)
    rows = np.concatenate([rng.choice(np.nonzero(mask_np & (tok_model == k))[0], n_sample, replace=False)
                           for k in range(K)])
    hid = DeviceRows(w.hidden)
    W_bits = [pu.bf16_bits(x) for x in w.W]
    args = (hid, W_bits, w.cu_seqlens.numpy(), w.inv_role.numpy(), w.role_model.numpy(), w.target.numpy(),
            w.tok_mask.numpy())
    o = orc.ppo_loss_fwd_bwd(*args, old.cpu().numpy(), ref.cpu().numpy(), adv.cpu().numpy(), clip_lo=w.clip_lo,
                             clip_hi=w.clip_hi, kl_coef=w.kl_coef, kl_mode=w.kl_mode, ent_coef=w.ent_coef,
                             n_roles=w.n_roles, rows=rows, want_dW=False)
    idx = o["dh_index"]
    assert idx.size == rows.size
    for key in ("logp", "entropy", "tok_loss"):
        assert np.abs(gp[key].cpu().numpy()[idx] - o[key][idx]).max() <= pu.TOL_LOGP, key
    assert np.abs(gl["logp"].cpu().numpy()[idx] - o["logp"][idx]).max() <= pu.TOL_LOGP
    assert np.abs(gl["lse"].cpu().numpy()[idx] - o["lse"][idx]).max() <= pu.TOL_LOGP
    dh = gp["dHidden"][torch.as_tensor(idx, device="cuda")].float().cpu().numpy()
    assert pu.rel_fro(dh, o["dHidden"]) <= pu.TOL_GRAD
    slack = pu.dh_row_allowance(w, o, gp["logp"].cpu().numpy(), old.cpu().numpy(), ref.cpu().numpy(), adv.cpu().numpy())
    assert pu.worst_row_rel(dh, o["dHidden"], slack) <= pu.TOL_GRAD
    # masked rows are zero everywhere
    off = torch.as_tensor(np.nonzero(~mask_np)[0][:4096], device="cuda")
    assert torch.all(gp["dHidden"][off] == 0) and torch.all(gp["logp"][off] == 0)

    # ---- (ii) loss = sum of exported token losses / M_k
    tl = gp["tok_loss"].double().cpu().numpy()
    M = np.array([max(float((mask_np & (tok_model == k)).sum()), 1.0) for k in range(K)])
    assert np.array_equal(gp["metrics"][:K, 0].cpu().numpy(), M)
    for k in range(K):
        ref_loss = tl[mask_np & (tok_model == k)].sum() / M[k]
        assert abs(gp["loss"][k].item() - ref_loss) <= pu.TOL_LOSS * abs(ref_loss) + 1e-7

    # ---- (iii) dW: column sums vanish; one row chunk checked in full with the full-batch norm; additivity
    for k in range(K):
        g = gp["dW"][k].double()
        assert g.sum(0).abs().max().item() <= 1e-2 * g.abs().sum(0).max().item()
    # one chunk of consecutive valid rows PER MODEL, all run in one call (a model's dW sees only its own chunk)
    chunks = []
    for k in range(K):
        cand = np.nonzero(mask_np & (tok_model == k))[0]
        start = int(rng.integers(0, cand.size - chunk_rows))
        chunks.append(cand[start:start + chunk_rows])
    chunk = np.concatenate(chunks)
    mask_c = np.zeros(n, np.uint8)
    mask_c[chunk] = 1
    d.tok_mask = torch.from_numpy(mask_c).cuda()
    dW_c = [torch.zeros(w.V, w.H, device="cuda") for _ in range(K)]
    gc = pu.gpu_ppo(ctx, w, d, old, ref, adv, norm=M.tolist(), dW=dW_c)
    for k in range(K):                       # the oracle takes one model at a time (an fp64 dW is several GB)
        oc = orc.ppo_loss_fwd_bwd(*args, old.cpu().numpy(), ref.cpu().numpy(), adv.cpu().numpy(),
                                  clip_lo=w.clip_lo, clip_hi=w.clip_hi, kl_coef=w.kl_coef, kl_mode=w.kl_mode,
                                  ent_coef=w.ent_coef, n_roles=w.n_roles, norm=M.tolist(), dW_models=[k],
                                  rows=chunks[k])
        assert np.array_equal(oc["dh_index"], chunks[k])
        got = dW_c[k].cpu().numpy()
        assert pu.rel_fro(got, oc["dW"][k]) <= pu.TOL_GRAD, k
        assert pu.worst_block_rel_fro(got, oc["dW"][k]) <= pu.TOL_GRAD, k      # per tile of 256 vocabulary rows
        rows_k = torch.as_tensor(chunks[k], device="cuda")
        slack = pu.dh_row_allowance(w, oc, gc["logp"].cpu().numpy(), old.cpu().numpy(), ref.cpu().numpy(),
                                    adv.cpu().numpy())
        assert pu.worst_row_rel(gc["dHidden"][rows_k].float().cpu().numpy(), oc["dHidden"], slack) <= pu.TOL_GRAD, k
        del oc, got
    # the rest of the batch accumulated on top of the chunk reproduces the full-batch dW
    mask_rest = w.tok_mask.clone()
    mask_rest[torch.from_numpy(chunk)] = 0
    d.tok_mask = mask_rest.cuda()
    pu.gpu_ppo(ctx, w, d, old, ref, adv, norm=M.tolist(), accumulate=True, dW=dW_c)
    for k in range(K):
        num = (dW_c[k] - gp["dW"][k]).double().norm().item()
        den = gp["dW"][k].double().norm().item()
        assert num <= 1e-3 * den
    ctx.close()
