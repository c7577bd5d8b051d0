"""apollo_mini_step_static -- the rank-1 step that allocates nothing -- against apollo_step.

Some users of this library cannot allocate device memory when the optimizer has to run
(a plug-in inside another runtime's memory plan, a loop that must not pay the
synchronisation of an allocation, a process whose pool is fully handed out), so they
cannot give apollo_create a workspace.  For them the library carries a fixed scratch array
and one entry point that uses it.  This test drives that entry point through the C ABI on
two steps in a row and checks weights, moments and limiter norm against the regular
context-based step on the same inputs, then against the CPU oracle, and checks that the
device's free memory does not move across a call.  It lives in a file that is collected
last, so a run that stops at the first failure has already run every other test.
"""
import math

import numpy as np
import pytest
import torch

from paper_2412_05270_b200 import binding as B
from paper_2412_05270_b200 import workloads as WL
from parity import DW_ABS, DW_REL, _f32, oracle_of

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("shape,dtype,mode", [
    ((1100, 1300), "bf16", "tensor"),     # wide, several row slices and column tiles
    ((1300, 520), "bf16", "tensor"),      # tall
    ((257, 1029), "f32", "channel"),      # unaligned pitch, scalar loads
    ((264, 1029), "bf16", "tensor"),      # unaligned pitch, rows a multiple of 8: update pass over groups of eight rows
])
def test_two_consecutive_static_steps_match_the_context_step(shape, dtype, mode):
    dev = torch.device("cuda")
    wl = WL.Workload("static", [shape], dtype, 1, mode, T=1, steps=2, wd=0.01,
                     alpha=math.sqrt(128.0) if mode == "tensor" else 1.0)
    cfg = B.config_for(wl)
    n = max(shape)
    W_ref = WL.make_weight(wl, 0).to(dev)
    W_sta = W_ref.clone()
    M = torch.zeros(n, dtype=torch.float32, device=dev)
    V = torch.zeros(n, dtype=torch.float32, device=dev)
    prev = torch.zeros(1, dtype=torch.float32, device=dev)
    # leave junk in front of the second case on purpose: an earlier call's contents must not matter
    opt = B.Apollo([shape], cfg)
    for t in range(2):
        G = WL.make_grad(wl, 0, t).to(dev)
        W_before = W_ref.float().clone()
        opt.step([W_ref], [G], wl.lr, wl.wd)
        B.mini_step_static(W_sta, G, M, V, prev, cfg, matrix=0, t=t, lr=wl.lr, wd=wl.wd)
        torch.cuda.synchronize()
        M_ref, V_ref = opt.state(0)
        lim = opt.limiter(0)
        torch.cuda.synchronize()
        # same kernels, same order of operations: the tolerance of the parity tests
        # (2e-3 of the largest update) is met with room to spare; in practice bit-equal
        bound = 2e-3 * (W_ref.float() - W_before).abs().max().item() + 1e-6
        assert (W_ref.float() - W_sta.float()).abs().max().item() <= bound
        assert torch.equal(W_ref, W_sta)
        assert torch.allclose(M, M_ref[0], rtol=1e-6, atol=0)
        assert torch.allclose(V, V_ref[0], rtol=1e-6, atol=0)
        assert abs(prev.item() - lim[0].item()) <= 1e-6 * abs(lim[0].item())
    assert opt.status() == B.OK
    opt.close()


@pytest.mark.parametrize("shape,mode", [((520, 1300), "tensor"), ((1300, 520), "channel")])
def test_static_steps_against_the_oracle(shape, mode):
    """Five steps across a projection refresh (T = 3), the caller keeping t, M, V and the previous
    norm: the weights follow the oracle's within the parity bound on the update."""
    dev = torch.device("cuda")
    wl = WL.Workload("static_oracle", [shape], "bf16", 1, mode, T=3, steps=5, wd=0.01,
                     alpha=math.sqrt(128.0) if mode == "tensor" else 1.0)
    cfg = B.config_for(wl)
    n = max(shape)
    W = WL.make_weight(wl, 0).to(dev)
    M = torch.zeros(n, dtype=torch.float32, device=dev)
    V = torch.zeros(n, dtype=torch.float32, device=dev)
    prev = torch.zeros(1, dtype=torch.float32, device=dev)
    orc = oracle_of(wl, [0])[0]
    Wo = W.float().cpu().numpy()
    for t in range(wl.steps):
        G = WL.make_grad(wl, 0, t).to(dev)
        B.mini_step_static(W, G, M, V, prev, cfg, matrix=0, t=t, lr=wl.lr, wd=wl.wd)
        torch.cuda.synchronize()
        res = orc.step(Wo, G.float().cpu().numpy(), _f32(wl.lr), _f32(wl.wd))
        bound = DW_REL * np.max(np.abs(res.dW)) + DW_ABS
        # the stored weight is a bf16 rounding of W_old + dW: one rounding step of slack on top of the bound
        tol = 2.0 ** -7 * np.abs(res.W) + bound
        assert np.all(np.abs(W.float().cpu().numpy() - res.W) <= tol), f"step {t}"
        assert abs(prev.item() - res.norm) <= 2e-3 * res.norm
        np.testing.assert_allclose(M.cpu().numpy(), orc.M[0], rtol=2e-3, atol=2e-3 * np.abs(orc.M).max())
        Wo = res.W
        W.copy_(torch.from_numpy(res.W).to(W.dtype))     # keep the two trajectories on the same weights


def test_a_static_step_obtains_no_device_memory():
    dev = torch.device("cuda")
    shape = (640, 1024)
    wl = WL.Workload("static_mem", [shape], "bf16", 1, "tensor", T=1, steps=2, alpha=math.sqrt(128.0))
    cfg = B.config_for(wl)
    W = WL.make_weight(wl, 0).to(dev)
    G = WL.make_grad(wl, 0, 0).to(dev)
    M = torch.zeros(1024, dtype=torch.float32, device=dev)
    V = torch.zeros(1024, dtype=torch.float32, device=dev)
    prev = torch.zeros(1, dtype=torch.float32, device=dev)
    B.mini_step_static(W, G, M, V, prev, cfg, matrix=0, t=0, lr=wl.lr)      # first call on the device: looks the array up
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info(dev)
    B.mini_step_static(W, G, M, V, prev, cfg, matrix=0, t=1, lr=wl.lr)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info(dev)
    assert free_after == free_before


def test_oversized_and_wrong_rank_requests_are_rejected():
    dev = torch.device("cuda")
    small = torch.zeros(8, 8, dtype=torch.bfloat16, device=dev)
    f = torch.zeros(8, dtype=torch.float32, device=dev)
    cfg = B.make_config(rank=1, mode=B.SCALE_TENSOR)
    lib = B.load()
    # 65536 x 65536 would need 4n + 8n*128 bytes of temporaries: far above the 8 MiB array
    rc = lib.apollo_mini_step_static(small.data_ptr(), small.data_ptr(), 65536, 65536, f.data_ptr(), f.data_ptr(),
                                     f.data_ptr(), cfg, 0, 0, 0.1, 0.0, None)
    assert rc == B.ERR_TOO_LARGE
    cfg2 = B.make_config(rank=2)
    rc = lib.apollo_mini_step_static(small.data_ptr(), small.data_ptr(), 8, 8, f.data_ptr(), f.data_ptr(),
                                     f.data_ptr(), cfg2, 0, 0, 0.1, 0.0, None)
    assert rc == B.ERR_RANK
    # the moments of this entry point are floats: a request for two-byte moments is refused, not overrun
    cfg3 = B.make_config(rank=1, mode=B.SCALE_TENSOR, flags=B.FLAG_BF16_STATES)
    rc = lib.apollo_mini_step_static(small.data_ptr(), small.data_ptr(), 8, 8, f.data_ptr(), f.data_ptr(),
                                     f.data_ptr(), cfg3, 0, 0, 0.1, 0.0, None)
    assert rc == B.ERR_INVALID_ARG
    torch.cuda.synchronize()
