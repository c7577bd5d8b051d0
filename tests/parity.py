"""Shared driver of the parity tests: runs the CUDA library and the CPU oracle on the same
seeded inputs and compares them under the stated bounds.

Bounds: Philox draws bit-exact; per element |dW_gpu - dW_oracle| <= 2e-3 max|dW_oracle| + 1e-6;
scales within 1e-3 relative; stored W equal to round(W_old + dW_gpu) exactly.

The scale bound is stated against the projection in the precision of the GEMM operands: for
bfloat16 gradients at rank > 1 the oracle rounds the standard normals behind P to bfloat16, as
the tensor cores see them (against an unrounded P the scales move by up to 2.6e-3, which the
1e-3 bound does not allow).

Below rank 16 a channel's "norm" is the norm of very few numbers (one signed number at rank 1)
and can come out far below its typical size; such a channel's scale is a ratio of two nearly
cancelled sums and has no 1e-3 relative meaning in fp32.  Those channels are exempt from the
scale bound (never from the dW bound); the exempt fraction is returned in `worst["exempt"]`
and must stay below EXEMPT_MAX_LOW_RANK (or two channels, for matrices of fewer than 40).
From rank 16 on no channel is exempt.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2412_05270_b200 import binding as B
from paper_2412_05270_b200 import workloads as WL

DW_REL, DW_ABS, SCALE_REL = 2e-3, 1e-6, 1e-3
EXEMPT_BELOW = 0.02          # a channel is ill-conditioned when |R_j| or |R~_j| is under 2 % of the median
EXEMPT_RANK = 16             # ranks from here on: no exemption
EXEMPT_MAX_LOW_RANK = 0.05   # largest exempt fraction accepted below EXEMPT_RANK (rank 1: about 2 %)


def config_of(wl: WL.Workload, flags=0, bias_correction=False) -> B.Config:
    return B.config_for(wl, flags, bias_correction)


def _f32(x) -> float:
    """The value the C ABI's float field holds: both sides get the same configuration."""
    return float(np.float32(x))


def oracle_of(wl: WL.Workload, mats=None, bias_correction=False, state_bf16=False):
    mats = range(len(wl.shapes)) if mats is None else mats
    # P has the precision of the projection's operands: bfloat16 for bf16 gradients at rank > 1
    # (tensor-core operands), fp32 for fp32 gradients and for the rank-1 matrix-vector pass.
    p_bf16 = wl.dtype == "bf16" and wl.rank > 1
    return {i: oracle.MatrixOracle(wl.shapes[i][0], wl.shapes[i][1], rank=wl.rank,
                                   mode=oracle.MODE_TENSOR if wl.mode == "tensor" else oracle.MODE_CHANNEL,
                                   dtype=oracle.DT_BF16 if wl.dtype == "bf16" else oracle.DT_F32,
                                   seed=wl.seed, matrix_id=i, T=wl.T, alpha=_f32(wl.alpha), gamma=_f32(wl.gamma),
                                   beta1=_f32(wl.beta1), beta2=_f32(wl.beta2), eps=_f32(wl.eps),
                                   bias_correction=bias_correction, p_round_bf16=p_bf16, state_bf16=state_bf16)
            for i in mats}


def run_parity(wl: WL.Workload, steps=None, flags=0, bias_correction=False, check_mats=None, expect_path=None,
               grad_fn=None, gen_device="cpu", tuning=None):
    """Steps the whole list on the GPU and the matrices in `check_mats` on the oracle.

    With gen_device="cuda" the inputs are drawn on the GPU (large lists) and only the checked
    matrices are copied to the host for the oracle."""
    steps = wl.steps if steps is None else steps
    n = len(wl.shapes)
    check_mats = list(range(n)) if check_mats is None else list(check_mats)
    dev = torch.device("cuda")
    opt = B.Apollo(wl.shapes, config_of(wl, flags, bias_correction), tuning=tuning)
    if expect_path is not None:
        for i in check_mats:
            assert opt.path(i) == expect_path, (i, opt.path(i))
    Wg = [WL.make_weight(wl, i, device=gen_device).to(dev) for i in range(n)]
    deltas = [torch.zeros(wl.shapes[i], dtype=torch.float32, device=dev) if i in check_mats else None
              for i in range(n)]
    opt.set_delta_out(deltas)
    orc = oracle_of(wl, check_mats, bias_correction, state_bf16=bool(flags & B.FLAG_BF16_STATES))
    Wo = {i: Wg[i].float().cpu().numpy() for i in check_mats}
    worst = {"dw": 0.0, "s": 0.0, "exempt": 0.0}
    for t in range(steps):
        Gg = [(grad_fn(wl, i, t) if grad_fn else WL.make_grad(wl, i, t, device=gen_device)).to(dev)
              for i in range(n)]
        W_before = {i: Wg[i].clone() for i in check_mats}
        opt.step(Wg, Gg, wl.lr, wl.wd)
        assert opt.status() == B.OK
        for i in check_mats:
            res = orc[i].step(Wo[i], Gg[i].float().cpu().numpy(), _f32(wl.lr), _f32(wl.wd), want_R=True)
            dw_gpu = deltas[i].cpu().numpy().astype(np.float64)
            bound = DW_REL * np.max(np.abs(res.dW)) + DW_ABS
            err = np.max(np.abs(dw_gpu - res.dW))
            assert err <= bound, f"step {t} matrix {i}: |dW error| {err:.3e} > {bound:.3e}"
            worst["dw"] = max(worst["dw"], err / bound)
            s_gpu = opt.scales(i).cpu().numpy().astype(np.float64)
            rn = np.linalg.norm(res.R, axis=0)
            tn = res.s * rn
            good = np.ones(rn.shape, dtype=bool)
            if wl.mode != "tensor" and wl.rank < EXEMPT_RANK:
                good = (rn >= EXEMPT_BELOW * np.median(rn)) & (tn >= EXEMPT_BELOW * np.median(tn))
            exempt = 1.0 - float(good.mean())
            assert (~good).sum() <= max(2, EXEMPT_MAX_LOW_RANK * good.size), \
                f"step {t} matrix {i}: {exempt:.3f} of the channels exempt"
            worst["exempt"] = max(worst["exempt"], exempt)
            rel = np.abs(s_gpu - res.s) / (np.abs(res.s) + 1e-30)
            assert np.all(rel[good] <= SCALE_REL), f"step {t} matrix {i}: scale rel error {rel[good].max():.3e}"
            worst["s"] = max(worst["s"], float(rel[good].max()))
            lim = opt.limiter(i).cpu().numpy()
            assert abs(lim[0] - res.norm) <= 2e-3 * res.norm + 1e-30
            assert abs(lim[1] - res.c) <= 2e-3
            # the store is exactly round(W_old + dW_gpu) in the weight's dtype
            want = (W_before[i].float() + deltas[i]).to(Wg[i].dtype)
            assert torch.equal(want, Wg[i]), f"step {t} matrix {i}: stored W is not round(W_old + dW)"
            # and agrees with the oracle's store up to one rounding step of the dtype
            w_gpu = Wg[i].float().cpu().numpy()
            tol = (2.0 ** -7 if wl.dtype == "bf16" else 1e-6) * np.abs(res.W) + bound
            assert np.all(np.abs(w_gpu - res.W) <= tol)
            Wo[i] = res.W
            # keep the two weight trajectories identical so that errors do not compound through wd
            Wg[i].copy_(torch.from_numpy(res.W).to(Wg[i].dtype))
        del Gg
    assert opt.step_count() == steps
    opt.close()
    return worst
