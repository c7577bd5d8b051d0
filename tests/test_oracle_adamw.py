"""Pins for the oracle's AdamW (the optimizer of the parameters APOLLO does not project):
torch.optim.AdamW as the library reference, and the printed Eq. 1 without bias correction."""
import numpy as np
import torch

import oracle


def test_matches_torch_adamw_over_several_steps():
    torch.manual_seed(0)
    p0 = torch.randn(257, dtype=torch.float64) * 0.1
    p = torch.nn.Parameter(p0.clone())
    opt = torch.optim.AdamW([p], lr=3e-3, betas=(0.9, 0.95), eps=1e-8, weight_decay=0.1)
    mine = p0.numpy().astype(np.float32)
    m = np.zeros(257); v = np.zeros(257)
    ref32 = torch.nn.Parameter(p0.float().clone())
    opt32 = torch.optim.AdamW([ref32], lr=3e-3, betas=(0.9, 0.95), eps=1e-8, weight_decay=0.1)
    for t in range(6):
        g = torch.randn(257, dtype=torch.float64).float()
        ref32.grad = g.clone()
        opt32.step()
        mine, _ = oracle.adamw_step(mine, g.numpy(), m, v, t, lr=3e-3, beta1=0.9, beta2=0.95, eps=1e-8, wd=0.1)
        np.testing.assert_allclose(mine, ref32.detach().numpy(), rtol=2e-5, atol=1e-7)


def test_without_bias_correction_is_the_printed_rule():
    g = np.array([0.5, -2.0, 0.0, 1e-3], dtype=np.float32)
    p = np.array([1.0, 1.0, 1.0, 1.0], dtype=np.float32)
    m = np.zeros(4); v = np.zeros(4)
    out, dp = oracle.adamw_step(p, g, m, v, 0, lr=0.1, beta1=0.9, beta2=0.999, eps=0.0, wd=0.0, bias_correction=False)
    # first step: m = 0.1 g, v = 0.001 g^2 -> m / sqrt(v) = sqrt(10) sign(g); g = 0 gives 0/0 -> nan is avoided by eps
    want = -0.1 * np.sqrt(10.0) * np.sign(g[[0, 1, 3]].astype(np.float64))
    np.testing.assert_allclose(dp[[0, 1, 3]], want, rtol=1e-6)
    np.testing.assert_allclose(m, 0.1 * g.astype(np.float64), rtol=1e-12)
    np.testing.assert_allclose(v, 0.001 * g.astype(np.float64) ** 2, rtol=1e-12)


def test_weight_decay_is_decoupled_and_bf16_store_rounds():
    p = np.array([0.3, -0.7], dtype=np.float32)
    m = np.zeros(2); v = np.zeros(2)
    out, dp = oracle.adamw_step(p, np.zeros(2, dtype=np.float32), m, v, 0, lr=0.1, eps=1e-8, wd=0.5)
    np.testing.assert_allclose(dp, -0.05 * p.astype(np.float64), rtol=1e-12)
    pb = torch.tensor([0.3, -0.7]).to(torch.bfloat16).float().numpy()
    outb, dpb = oracle.adamw_step(pb, np.array([1.0, 1.0], dtype=np.float32), np.zeros(2), np.zeros(2), 0, lr=1e-3,
                                  wd=0.0, dtype=oracle.DT_BF16)
    want = np.array([oracle.round_bf16(float(pb[i]) + dpb[i]) for i in range(2)])
    assert np.array_equal(outb.astype(np.float64), want)
