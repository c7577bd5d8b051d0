"""Parity on the LLaMA-shaped configurations, in the launch configuration the benchmark times.

Every list runs on the GPU in full for ten consecutive steps that include a projection refresh.
350M, 1B and 7B-Mini: a few matrices of every kind are stepped on the oracle in full.  7B at rank
256: the oracle re-computes sampled channels (a channel's scale, moments and update depend only
on that channel's column of G and on P, which depends on the row index alone), the square matrix
in full, and the limiter is checked through the identities Eq. 4 fixes.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2412_05270_b200 import binding as B
from paper_2412_05270_b200 import workloads as WL
from parity import DW_ABS, DW_REL, SCALE_REL, _f32, run_parity

pytestmark = pytest.mark.gpu


def test_llama350m_rank256_across_a_refresh():
    wl = WL.workload("llama350m")
    wl.T = 5
    # q (square), gate (wide, 2736 = 10 x 256 + 176 columns), down (tall), and the last matrix
    worst = run_parity(wl, steps=10, check_mats=[0, 4, 6, 167], expect_path=B.PATH_TENSOR, gen_device="cuda")
    assert worst["dw"] <= 1.0 and worst["exempt"] == 0.0


def test_llama1b_rank512_ten_steps_across_a_refresh():
    """The whole 168-matrix list on the GPU (rank 512, weight decay 0.01, outlier columns), ten
    consecutive steps with the projection refreshed at step 5; a square matrix, a 2048 x 5461 one
    (row pitch that is not a multiple of 16 bytes), a 5461 x 2048 one and the last matrix of the
    list are stepped on the oracle in full."""
    wl = WL.workload("llama1b")
    wl.T = 5
    opt_paths = B.Apollo(wl.shapes, B.config_for(wl))
    assert opt_paths.path(0) == B.PATH_TENSOR and opt_paths.path(6) == B.PATH_TENSOR
    assert opt_paths.path(4) == B.PATH_TENSOR  # 5461 columns
    opt_paths.close()
    worst = run_parity(wl, steps=10, check_mats=[0, 4, 6, 167], gen_device="cuda")
    assert worst["dw"] <= 1.0 and worst["exempt"] == 0.0


def test_llama1b_realigned_in_the_kernel():
    """The same list with the 2048 x 5461 gradients fetched as they lie and re-aligned in shared memory
    (apollo_tuning.realign = 1: no padded copies): six steps across a refresh, the two kinds of MLP matrices."""
    wl = WL.workload("llama1b")
    wl.T = 3
    worst = run_parity(wl, steps=6, check_mats=[4, 6], gen_device="cuda", tuning=B.make_tuning(realign=1))
    assert worst["dw"] <= 1.0 and worst["exempt"] == 0.0


def test_llama7b_mini_full_list_ten_steps_across_a_refresh():
    """All 224 matrices at rank 1 with the tensor-wise scale, ten consecutive steps with the
    projection refreshed at step 5; four matrices of every kind on the oracle in full."""
    wl = WL.workload("llama7b_mini")
    wl.T = 5
    worst = run_parity(wl, steps=10, check_mats=[0, 4, 6, 223], expect_path=B.PATH_STREAM, gen_device="cuda")
    assert worst["dw"] <= 1.0


def _sample(n, count, tile):
    """Channel sample: random, plus the first and last channels and both sides of tile boundaries."""
    g = np.random.default_rng(n)
    forced = {0, 1, n - 1, n - 2, tile - 1, tile, 2 * tile - 1, 2 * tile, (n // tile) * tile - 1, (n // tile) * tile}
    forced = sorted(j for j in forced if 0 <= j < n)
    others = np.setdiff1d(np.arange(n), np.array(forced))
    rest = g.choice(others, size=count - len(forced), replace=False)
    return np.sort(np.concatenate([np.array(forced, dtype=np.int64), rest.astype(np.int64)]))


def test_llama7b_full_list_sampled_channels_and_limiter():
    wl = WL.workload("llama7b")
    wl.T = 5
    dev = torch.device("cuda")
    n_mat = len(wl.shapes)
    steps = 10          # consecutive, with the projection refreshed at step 5
    lr, wd = _f32(wl.lr), _f32(wl.wd)
    opt = B.Apollo(wl.shapes, B.config_for(wl))
    checks = {0: None, 4: "cols", 6: "rows", 223: "rows"}      # q in full, gate by columns, down by rows
    for i in checks:
        assert opt.path(i) == B.PATH_TENSOR
    Wg = [WL.make_weight(wl, i, device=dev) for i in range(n_mat)]
    deltas = [torch.zeros(wl.shapes[i], dtype=torch.float32, device=dev) if i in checks else None for i in range(n_mat)]
    opt.set_delta_out(deltas)
    sel, orc, Wo = {}, {}, {}
    for i, kind in checks.items():
        rows, cols = wl.shapes[i]
        m, n = min(rows, cols), max(rows, cols)
        # keep the sub-problem's orientation: at least m columns for a wide matrix, m + 1 rows for a tall one
        sel[i] = None if kind is None else _sample(n, m if kind == "cols" else m + 1, 256)
        sub = (rows, cols) if kind is None else ((rows, len(sel[i])) if kind == "cols" else (len(sel[i]), cols))
        orc[i] = oracle.MatrixOracle(sub[0], sub[1], rank=wl.rank, mode=oracle.MODE_CHANNEL, dtype=oracle.DT_BF16,
                                     seed=wl.seed, matrix_id=i, T=wl.T, alpha=_f32(wl.alpha),
                                     gamma=_f32(wl.gamma) if kind is None else 0.0, beta1=_f32(wl.beta1),
                                     beta2=_f32(wl.beta2), eps=_f32(wl.eps), p_round_bf16=True)

    def sub_of(x, i):
        kind = checks[i]
        if kind is None:
            return x
        idx = torch.from_numpy(sel[i]).to(x.device)
        return x.index_select(1 if kind == "cols" else 0, idx)

    prev_norm = {i: 0.0 for i in checks}
    for t in range(steps):
        Gg = [WL.make_grad(wl, i, t, device=dev) for i in range(n_mat)]
        W_before = {i: Wg[i].clone() for i in checks}
        opt.step(Wg, Gg, wl.lr, wl.wd)
        assert opt.status() == B.OK
        for i, kind in checks.items():
            res = orc[i].step(sub_of(W_before[i], i).float().cpu().numpy(), sub_of(Gg[i], i).float().cpu().numpy(),
                              lr, wd)
            s_gpu_full = opt.scales(i)
            s_gpu = (s_gpu_full if kind is None else s_gpu_full[torch.from_numpy(sel[i]).to(dev)]).cpu().numpy().astype(np.float64)
            rel = np.abs(s_gpu - res.s) / np.abs(res.s)
            assert rel.max() <= SCALE_REL, f"step {t} matrix {i}: scale rel error {rel.max():.3e}"
            lim = opt.limiter(i).cpu().numpy().astype(np.float64)     # norm, c, raw norm, tensor scale
            # Eq. 4 through identities that hold at any size: the raw norm is |G diag(s)|_F, the factor
            # is gamma prev / raw when that ratio is exceeded and 1 otherwise, the kept norm is c raw
            g32 = Gg[i].float()
            scaled = g32 * (s_gpu_full[None, :] if wl.shapes[i][0] <= wl.shapes[i][1] else s_gpu_full[:, None])
            raw = float(torch.linalg.vector_norm(scaled.double()))
            assert abs(lim[2] - raw) <= 1e-4 * raw
            gamma = _f32(wl.gamma)
            want_c = gamma * prev_norm[i] / raw if (prev_norm[i] > 0 and raw > gamma * prev_norm[i]) else 1.0
            assert abs(lim[1] - want_c) <= 1e-4
            assert abs(lim[0] - want_c * raw) <= 1e-4 * raw
            if t > 0:
                assert lim[0] <= gamma * prev_norm[i] * (1 + 1e-5)
            prev_norm[i] = lim[0]
            # update of the sampled channels: the oracle's (limiter off) times the factor c
            c = lim[1] if kind is not None else 1.0
            dw_gpu = sub_of(deltas[i], i).cpu().numpy().astype(np.float64)
            dw_or = res.dW * c
            bound = DW_REL * np.max(np.abs(dw_or)) + DW_ABS
            err = np.max(np.abs(dw_gpu - dw_or))
            assert err <= bound, f"step {t} matrix {i}: |dW error| {err:.3e} > {bound:.3e}"
            if kind is None:
                assert abs(lim[1] - res.c) <= 2e-3 and abs(lim[0] - res.norm) <= 2e-3 * res.norm
            want = (W_before[i].float() + deltas[i]).to(torch.bfloat16)
            assert torch.equal(want, Wg[i])
            # moments of the sampled channels (a bf16 rounding of one entry of P that falls the other way on
            # the GPU moves one term by 2^-8: entries near zero get the absolute allowance)
            M, V = opt.state(i)
            idx = slice(None) if kind is None else torch.from_numpy(sel[i]).to(dev)
            np.testing.assert_allclose(M[:, idx].cpu().numpy(), orc[i].M, rtol=2e-3, atol=5e-3 * np.median(np.abs(orc[i].M)))
            np.testing.assert_allclose(V[:, idx].cpu().numpy(), orc[i].V, rtol=4e-3, atol=5e-3 * np.median(np.abs(orc[i].V)))
        del Gg
    opt.close()


def test_matrix_with_more_than_2_31_elements_rank1():
    """Flat indices above 2^31: 70000 x 32768 bf16 (2.29 G elements), Mini step checked with torch on the
    GPU (the generator itself is pinned bit-exactly against the oracle elsewhere)."""
    dev = torch.device("cuda")
    rows, cols = 70000, 32768
    assert rows * cols > 2 ** 31
    g = torch.Generator(device=dev).manual_seed(11)
    W = torch.empty(rows, cols, dtype=torch.bfloat16, device=dev).normal_(0, 0.02, generator=g)
    G = torch.empty(rows, cols, dtype=torch.bfloat16, device=dev).normal_(0, 1e-3, generator=g)
    W0_tail = W[-3:].float().clone()
    W0_head = W[:2].float().clone()
    alpha = math.sqrt(128.0)
    cfg = B.make_config(rank=1, mode=B.SCALE_TENSOR, dtype=B.DT_BF16, T=5, seed=77, alpha=alpha, gamma=1.01)
    opt = B.Apollo([(rows, cols)], cfg)
    assert opt.path(0) == B.PATH_STREAM
    opt.step([W], [G], 1e-2, 0.0)
    torch.cuda.synchronize()
    assert opt.status() == B.OK
    # tall matrix: project along the 32768 columns, one channel per row
    z = B.projection(77, 0, 0, 1, cols)[0].double()
    R = torch.empty(rows, dtype=torch.float64, device=dev)
    for a in range(0, rows, 10000):
        R[a:a + 10000] = G[a:a + 10000].double() @ z
    Rt = (0.1 * R) / (torch.sqrt(0.001 * R * R) + 1e-8)
    s_want = (Rt.norm() / R.norm()).item()
    s_gpu = opt.scales(0)
    assert torch.all(s_gpu == s_gpu[0])
    assert abs(s_gpu[0].item() - s_want) <= 1e-4 * s_want
    lim = opt.limiter(0).cpu().numpy()
    g_norm = math.sqrt(sum(float(G[a:a + 10000].float().square().sum()) for a in range(0, rows, 10000)))
    assert abs(lim[2] - s_want * g_norm) <= 1e-3 * s_want * g_norm and lim[1] == 1.0
    M, V = opt.state(0)
    assert torch.allclose(M[0].double(), 0.1 * R, rtol=1e-3, atol=1e-3 * float(R.abs().median()) * 0.1)
    # the update at the very end of the flat array (indices above 2^31) and at its start
    step = 1e-2 * alpha * s_gpu[0].item()
    for sl, before in ((slice(rows - 3, rows), W0_tail), (slice(0, 2), W0_head)):
        want = (before - step * G[sl].float()).to(torch.bfloat16)
        got = W[sl]
        assert (want.float() - got.float()).abs().max().item() <= 2.0 ** -7 * before.abs().max().item()
        assert (want == got).float().mean().item() > 0.99
    opt.close()


def test_one_by_one_matrix():
    dev = torch.device("cuda")
    opt = B.Apollo([(1, 1)], B.make_config(rank=1, mode=B.SCALE_CHANNEL, dtype=B.DT_F32, seed=3, gamma=0.0, eps=0.0))
    W = torch.tensor([[0.5]], device=dev)
    G = torch.tensor([[2.0]], device=dev)
    opt.step([W], [G], 0.1, 0.0)
    torch.cuda.synchronize()
    # R = z g, M = 0.1 R, V = 0.001 R^2 -> |R~| / |R| = sqrt(10) / |z g|; update = lr s g
    z = abs(B.projection(3, 0, 0, 1, 1).item())
    s = math.sqrt(10.0) / (z * 2.0)
    assert abs(opt.scales(0).item() - s) <= 1e-5 * s
    assert abs(W.item() - (0.5 - 0.1 * s * 2.0)) <= 1e-5
    opt.close()
