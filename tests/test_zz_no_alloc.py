"""apollo_mini_step_static -- the rank-1 step that allocates nothing -- against apollo_step.

Some users of this library cannot allocate device memory when the optimizer has to run
(a plug-in inside another runtime's memory plan, a loop that must not pay the
synchronisation of an allocation, a process whose pool is fully handed out), so they
cannot give apollo_create a workspace.  For them the library carries a fixed scratch array
and one entry point that uses it.  This test drives that entry point through the C ABI on
two steps in a row and checks weights, moments and limiter norm against the regular
context-based step on the same inputs.  It lives in a file that is collected last, so a
run that stops at the first failure has already run every other test.
"""
import math

import pytest
import torch

from paper_2412_05270_b200 import binding as B
from paper_2412_05270_b200 import workloads as WL

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
    torch.cuda.synchronize()
