"""The bounded-wait exit of the GEMM kernels, exercised in its host-visible form.

Every in-kernel wait (on a shared-memory stage, an accumulator stage, the peer CTA) carries a clock budget.  Here the
budget is set to 400 000 SM clocks and a test hook makes the TMA producer of one GEMM class leave out a single K slab
of every worker's first tile: the MMA issuer's wait for that slab runs out, the other roles' waits behind it run out in
turn, every role of both CTAs leaves its loop, tensor memory is freed and the launch returns within milliseconds.
Nothing faults, traps or spins without limit.  The host must see UNITY_ERR_TIMEOUT, and the same context must then
compute a normal call correctly."""
import time

import numpy as np
import pytest
import torch

import parity_harness as pu
from paper_2605_26646_b200 import binding as ub
from paper_2605_26646_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("ctas", [1, 2])
@pytest.mark.parametrize("cls", ["fwd_gemm", "grad_gemm", "dh_gemm", "dw_gemm"])
def test_expired_wait_reports_timeout_and_context_stays_usable(cls, ctas):
    w = wl.make("tiny", device="cuda")
    d = pu.DeviceInputs(w)
    ctx = pu.make_ctx(w)
    for option in range(4):
        ctx.set_option(option, ctas)
    # the hook is refused while the wait bound is long
    with pytest.raises(ub.UnityError) as e:
        ctx.set_option(ub.OPT_TEST_DROP_SLAB, 1)
    assert e.value.code == -1
    ol, oa = pu.oracle_logprob(w), pu.oracle_advantage(w)
    cur = torch.from_numpy(ol["logp"].astype(np.float32))
    old, ref = (cur + w.noise_old).cuda(), (cur + w.noise_ref).cuda()
    adv = torch.from_numpy(oa["adv_tok"].astype(np.float32)).cuda()

    ctx.set_option(ub.OPT_WAIT_KCYCLES, 400)
    ctx.set_option(ub.OPT_TEST_DROP_SLAB, 1 + ub.OPT_CTAS[cls])
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    with pytest.raises(ub.UnityError) as e:
        if cls == "fwd_gemm":
            pu.gpu_logprob(ctx, w, d)
        else:
            pu.gpu_ppo(ctx, w, d, old, ref, adv)
    assert e.value.code == -8, e.value
    assert time.perf_counter() - t0 < 2.0                      # milliseconds on the device; generous for the host
    # a longer bound switches the hook off by itself; the status was cleared by the check above
    ctx.set_option(ub.OPT_WAIT_KCYCLES, 4_000_000)
    ctx.check_status()
    gl = pu.gpu_logprob(ctx, w, d)
    assert np.abs(gl["logp"].cpu().numpy() - ol["logp"]).max() <= pu.TOL_LOGP
    gp = pu.gpu_ppo(ctx, w, d, old, ref, adv)
    op = pu.oracle_ppo(w, old.cpu().numpy(), ref.cpu().numpy(), adv.cpu().numpy())
    assert np.all(np.abs(gp["loss"].cpu().numpy() - op["loss"]) <= pu.TOL_LOSS * np.abs(op["loss"]) + 1e-7)
    assert pu.rel_fro(gp["dHidden"].float().cpu().numpy(), op["dHidden"]) <= pu.TOL_GRAD
    assert pu.rel_fro(gp["dW"][0].cpu().numpy(), op["dW"][0]) <= pu.TOL_GRAD
    ctx.close()
