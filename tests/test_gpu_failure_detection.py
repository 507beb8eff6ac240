"""A bounded device wait that runs out (the library's only failure signal on the device: no trap, no hang).

im_debug_set_wait shortens the limit to 1 ms and makes the copy-issuing threads idle, so the consumers of the
GEMM pipeline (and of the PPO loss kernel's tile pipeline) wait on a barrier that nothing will complete, with
no copy or MMA in flight.  The kernel must give up, report IM_DEV_WAIT_TIMEOUT (the loss: a NaN summary), return,
and leave the context usable: the next normal launch on the same buffers is correct."""
import numpy as np
import pytest
import torch

from paper_2609_09821_b200 import binding as B
from paper_2609_09821_b200 import workloads as W

pytestmark = pytest.mark.gpu

IM_DEV_WAIT_TIMEOUT = 2


@pytest.fixture
def short_wait_without_loads():
    B.debug_set_wait(1_000_000, True)            # 1 ms, producers idle
    try:
        yield
    finally:
        B.debug_set_wait()                       # back to 2 s, producers on


def _gemm_inputs():
    g = np.random.default_rng(0)
    a = W.round_to_bf16(g.standard_normal((64, 64)).astype(np.float32))[0]
    b = W.round_to_bf16((g.standard_normal((64, 64)) / 8).astype(np.float32))[0]
    A_, B_ = torch.from_numpy(a).cuda().to(torch.bfloat16), torch.from_numpy(b).cuda().to(torch.bfloat16)
    return a, b, A_, B_


def test_gemm_wait_runs_out_and_the_next_launch_is_correct(short_wait_without_loads):
    a, b, A_, B_ = _gemm_inputs()
    C_ = torch.full((64, 64), 9.0, dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    bias = torch.zeros(64, device="cuda")
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    B.gemm_bf16(A_, B_, C_, bias, False, status)
    t1.record()
    torch.cuda.synchronize()                     # the call returned and the kernel ended by itself
    assert status.item() & IM_DEV_WAIT_TIMEOUT
    assert t0.elapsed_time(t1) < 200.0           # milliseconds: the 1 ms limit, not the 2 s default
    B.debug_set_wait()
    status.zero_()
    B.gemm_bf16(A_, B_, C_, bias, False, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    want = a.astype(np.float64) @ b.astype(np.float64).T
    assert np.abs(C_.float().cpu().numpy() - want).max() <= 2.0 ** -8 * np.abs(want).max() + 1e-3


def test_ppo_loss_wait_runs_out_and_the_next_launch_is_correct(short_wait_without_loads):
    from oracle import oracle as O
    M, A = 64, 28
    pb_np = W.make_ppo_batch(M, A, 3, drift=0.02)
    pb = {k: torch.from_numpy(v).cuda() for k, v in pb_np.items()}
    ws = B.ppo_workspace()
    outs = [torch.zeros((M, A), device="cuda"), torch.zeros(A, device="cuda"), torch.zeros(M, device="cuda"),
            torch.zeros(6, device="cuda")]
    B.ppo_loss(pb, *outs, ws, 0.2, 2.0, 2.5e-4, True)
    torch.cuda.synchronize()
    assert torch.isnan(outs[3][0])               # the summary says the tiles never arrived
    B.debug_set_wait()
    B.ppo_loss(pb, *outs, ws, 0.2, 2.0, 2.5e-4, True)
    torch.cuda.synchronize()
    want = O.ppo_loss(pb_np, 0.2, 2.0, 2.5e-4, True)
    np.testing.assert_allclose(outs[3].cpu().numpy()[:4], want["summary"][:4], rtol=2e-4, atol=2e-5)
    assert torch.isfinite(outs[0]).all()
