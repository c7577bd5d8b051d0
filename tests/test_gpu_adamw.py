"""Fused AdamW (parameters APOLLO does not project) against the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2412_05270_b200 import binding as B

pytestmark = pytest.mark.gpu

SIZES = [1, 7, 8, 9, 1000, 8192, 8193, 70001, 4096 * 32] + [33 + 17 * i for i in range(30)]   # 39 tensors: two launches


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("bias_correction", [True, False])
def test_adamw_matches_the_oracle(dtype, bias_correction):
    dev = torch.device("cuda")
    g = torch.Generator().manual_seed(5)
    P = [(torch.randn(n, generator=g) * 0.05).to(dtype) for n in SIZES]
    Pg = [p.to(dev) for p in P]
    Ms = [torch.zeros(n, dtype=torch.float32, device=dev) for n in SIZES]
    Vs = [torch.zeros(n, dtype=torch.float32, device=dev) for n in SIZES]
    Ds = [torch.zeros(n, dtype=torch.float32, device=dev) for n in SIZES]
    Po = [p.float().numpy() for p in P]
    Mo = [np.zeros(n) for n in SIZES]
    Vo = [np.zeros(n) for n in SIZES]
    f32 = lambda x: float(np.float32(x))
    lr, b1, b2, eps, wd = f32(3e-3), f32(0.9), f32(0.95), f32(1e-8), f32(0.1)
    for t in range(4):
        G = [(torch.randn(n, generator=g) * 1e-2).to(dtype) for n in SIZES]
        before = [p.clone() for p in Pg]
        B.adamw_step(Pg, [x.to(dev) for x in G], Ms, Vs, t, lr, b1, b2, eps, wd, bias_correction, deltas=Ds)
        torch.cuda.synchronize()
        for i, n in enumerate(SIZES):
            out, dp = oracle.adamw_step(Po[i], G[i].float().numpy(), Mo[i], Vo[i], t, lr, b1, b2, eps, wd,
                                        dtype=oracle.DT_BF16 if dtype == torch.bfloat16 else oracle.DT_F32,
                                        bias_correction=bias_correction)
            d_gpu = Ds[i].cpu().numpy().astype(np.float64)
            assert np.max(np.abs(d_gpu - dp)) <= 2e-5 * np.max(np.abs(dp)) + 1e-9, (t, i)
            assert torch.equal((before[i].float() + Ds[i]).to(dtype), Pg[i])
            np.testing.assert_allclose(Ms[i].cpu().numpy(), Mo[i], rtol=1e-5, atol=1e-9)
            np.testing.assert_allclose(Vs[i].cpu().numpy(), Vo[i], rtol=1e-5, atol=1e-12)
            Po[i] = out
            Pg[i].copy_(torch.from_numpy(out).to(dtype))


def test_adamw_rejects_bad_arguments():
    dev = torch.device("cuda")
    p = torch.zeros(16, device=dev); m = torch.zeros(16, device=dev)
    with pytest.raises(B.ApolloError) as e:
        B.adamw_step([p], [p], [m], [m], 0, 1e-3, beta1=1.0)
    assert e.value.code == B.ERR_INVALID_ARG
    q = torch.zeros(20, device=dev)[1:17]          # 4-byte offset
    with pytest.raises(B.ApolloError) as e:
        B.adamw_step([q], [p], [m], [m], 0, 1e-3)
    assert e.value.code == B.ERR_ALIGN
