"""Parity of the CUDA step with the CPU oracle, element by element, through the C ABI."""
import dataclasses
import math

import pytest
import torch

from paper_2412_05270_b200 import binding as B
from paper_2412_05270_b200 import workloads as WL
from parity import run_parity

pytestmark = pytest.mark.gpu


def _wl(shapes, rank, mode="channel", dtype="bf16", T=3, steps=6, **kw):
    return WL.Workload("case", list(shapes), dtype, rank, mode, T=T, steps=steps, **kw)


SMALL = [(5, 7), (7, 5), (33, 130), (130, 33), (64, 64), (100, 257), (257, 100), (1, 9), (9, 1)]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("mode", ["channel", "tensor"])
def test_rank1_streaming_path_small_shapes(dtype, mode):
    wl = _wl(SMALL, 1, mode=mode, dtype=dtype, alpha=math.sqrt(128.0) if mode == "tensor" else 1.0, wd=0.05)
    run_parity(wl, expect_path=B.PATH_STREAM)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("rank,mode", [(2, "channel"), (5, "channel"), (5, "tensor")])
def test_cuda_core_path_small_shapes(dtype, rank, mode):
    shapes = [s for s in SMALL if min(s) >= rank]
    wl = _wl(shapes, rank, mode=mode, dtype=dtype, wd=0.05)
    run_parity(wl, flags=B.FLAG_NO_TENSOR_CORES, expect_path=B.PATH_SIMT)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_update_pass_over_groups_of_eight_rows_when_rows_are_not_whole_vectors(dtype):
    # wide, cols % 8 != 0, rows % 8 == 0: the update pass tiles 8-row groups (one group, a ragged last
    # tile of groups, several column chunks, columns that wrap inside a thread's eight elements)
    wl = _wl([(8, 9), (16, 37), (40, 2053), (136, 4099), (264, 333)], 2, dtype=dtype, wd=0.05, steps=4, T=2)
    run_parity(wl, flags=B.FLAG_NO_TENSOR_CORES, expect_path=B.PATH_SIMT)


def test_cuda_core_path_rank_spanning_row_blocks_and_ragged_tiles():
    wl = _wl([(200, 333), (333, 200), (130, 130)], 130, dtype="bf16", steps=4, T=2)
    run_parity(wl, flags=B.FLAG_NO_TENSOR_CORES, expect_path=B.PATH_SIMT)


def test_streaming_path_spanning_row_blocks_and_column_tiles():
    # wide: > 512 rows and > 256 columns with ragged tails; tall: > 2048 columns of P per chunk
    wl = _wl([(1100, 1300), (1300, 1100), (600, 2600), (70, 3000), (3000, 2100)], 1, mode="tensor", dtype="bf16",
             steps=3, alpha=math.sqrt(128.0))
    run_parity(wl, expect_path=B.PATH_STREAM)
    # unaligned pitch (scalar loads).  Tensor-wise scale: at rank 1 a channel-wise scale divides by
    # one signed number per channel, which among a thousand channels cancels to ~1e-4 of its terms
    # somewhere, and no fp32 path can then hold a relative bound.
    wl = _wl([(1029, 1301), (1301, 1029)], 1, mode="tensor", dtype="f32", steps=3, alpha=math.sqrt(128.0))
    run_parity(wl, expect_path=B.PATH_STREAM)


@pytest.mark.parametrize("rank,shapes", [
    (16, [(64, 72), (72, 64), (128, 128), (16, 520)]),
    (64, [(200, 1000), (1000, 200), (520, 264)]),
    (128, [(300, 1032), (1032, 304)]),
    (256, [(512, 1376), (1376, 512), (512, 512)]),
    (512, [(512, 1376), (1376, 512)]),
    (48, [(96, 200), (200, 96)]),
    # row pitch not a multiple of 16 bytes.  Wide with rows % 8 == 0: tiles fetched as they lie and re-aligned in
    # shared memory; tall, or rows % 8 != 0: padded copy.  Mixed with aligned matrices in one list.
    (32, [(200, 333), (336, 203), (64, 77)]),
    (64, [(264, 1029), (200, 1000), (200, 1001), (204, 333), (1000, 203)]),
    (256, [(512, 1381), (512, 1376), (256, 257)]),
    (512, [(512, 1381), (1376, 512), (512, 515)]),  # two row slices per channel tile
    # ranks that are not multiples of 16: the MMA works on the rank rounded up, with zero rows of P
    (17, [(64, 72), (72, 64), (17, 520)]),
    (130, [(300, 1032), (1032, 304), (130, 130)]),
    (300, [(512, 1376), (1376, 512)]),              # above 256: rounded up to 320, two row slices of 160
])
def test_tensor_core_path(rank, shapes):
    wl = _wl(shapes, rank, dtype="bf16", steps=4, T=2, wd=0.01)
    run_parity(wl, expect_path=B.PATH_TENSOR)
    if any(c % 8 for _, c in shapes):
        # the same list with the unaligned wide matrices re-aligned in shared memory instead of copied
        run_parity(wl, expect_path=B.PATH_TENSOR, tuning=B.make_tuning(realign=1))
        # and with a 1 MB buffer for the padded copies: the matrices share it group by group
        run_parity(wl, expect_path=B.PATH_TENSOR, tuning=B.make_tuning(repitch_mb=1))
        run_parity(wl, flags=B.FLAG_KEEP_P, expect_path=B.PATH_TENSOR, tuning=B.make_tuning(repitch_mb=1))


MODES = [
    # (flags, tuning of the mode, tuning of the run to compare bits with)
    (B.FLAG_KEEP_P, {}, None),                                    # every matrix keeps its P for the epoch
    (0, {"p_generator": 1}, {}),                                  # a separate kernel fills the scratch (one group here)
    (0, {"p_generator": 1, "scratch_mb": 1}, {}),                 # ... group by group: the scratch holds 1 MB
    (0, {"scratch_mb": 1}, {}),                                   # generator warps, ring of two slots
    (0, {"r_slice": 64}, {"r_slice": 64, "p_generator": 1}),      # four row slices of R per channel tile
    (0, {"kernel": B.TC_KERNEL_RING}, None),                      # single-CTA kernel, 256 channels x 256 rows per tile
    (0, {"kernel": B.TC_KERNEL_RING, "scratch_mb": 1}, {"kernel": B.TC_KERNEL_RING}),
    (B.FLAG_KEEP_P, {"kernel": B.TC_KERNEL_RING, "r_slice": 128, "nblk": 2}, None),
    (0, {"p_source": B.P_SHARED}, {"kernel": B.TC_KERNEL_RING}),  # P generated in shared memory by every CTA (ring kernel)
    (0, {"p_source": B.P_SHARED, "r_slice": 128, "nblk": 4}, {"kernel": B.TC_KERNEL_RING, "r_slice": 128, "nblk": 4}),
    (0, {"epi_prefetch": 0}, {}),                                 # no L2 prefetch of the moments in the epilogue
    (0, {"epi_prefetch": 8, "r_slice": 64}, {"r_slice": 64}),     # prefetch distance beyond the chunks of a slice
]


@pytest.mark.parametrize("flags,mode,ref", MODES)
def test_tensor_core_path_selectable_modes(flags, mode, ref):
    """Every mode of the tensor path (apollo_tuning, APOLLO_FLAG_KEEP_P) meets the parity bounds, and since none
    of them changes P or, at equal tile shape, the order of any sum, it gives the same bits as the run it is
    paired with."""
    shapes = [(512, 1376), (1376, 512), (512, 512), (300, 1032), (1376, 1400)]   # P: 1.6 MB in all
    wl = _wl(shapes, 256, dtype="bf16", steps=4, T=2, wd=0.01)
    dev = torch.device("cuda")

    def final_weights(fl, tu):
        opt = B.Apollo(wl.shapes, B.config_for(wl, fl), tuning=B.make_tuning(**tu))
        W = [WL.make_weight(wl, i).to(dev) for i in range(len(shapes))]
        for t in range(4):
            opt.step(W, [WL.make_grad(wl, i, t).to(dev) for i in range(len(shapes))], wl.lr, wl.wd)
        assert opt.status() == B.OK
        out = W, [opt.scales(i) for i in range(len(shapes))]
        opt.close()
        return out

    run_parity(wl, flags=flags, expect_path=B.PATH_TENSOR, tuning=B.make_tuning(**mode))
    if ref is not None:
        W_ref, s_ref = final_weights(0, ref)
        W_mode, s_mode = final_weights(flags, mode)
        for a, b in zip(W_ref, W_mode):
            assert torch.equal(a, b)
        for a, b in zip(s_ref, s_mode):
            assert torch.equal(a, b)


def test_tensor_core_path_tensor_mode_and_bias_correction():
    wl = _wl([(256, 520), (520, 256)], 32, mode="tensor", dtype="bf16", steps=3, T=2)
    run_parity(wl, expect_path=B.PATH_TENSOR, bias_correction=True)


def test_bias_correction_variant():
    wl = _wl([(33, 130), (130, 33)], 4, dtype="f32", steps=4)
    run_parity(wl, flags=B.FLAG_NO_TENSOR_CORES, bias_correction=True)
    wl = _wl([(33, 130), (130, 33)], 1, dtype="bf16", mode="tensor", steps=4)
    run_parity(wl, bias_correction=True)


def test_limiter_engages_on_growing_gradients():
    wl = _wl([(40, 90), (90, 40)], 4, dtype="f32", steps=8, T=4)

    def grad(w, i, t):
        return WL.make_grad(w, i, t) * (1.5 ** t)
    worst = run_parity(wl, flags=B.FLAG_NO_TENSOR_CORES, grad_fn=grad)
    assert worst["dw"] <= 1.0


def test_config_single_matrix_fp32_rank128():
    """fp32 gradients run on the tensor cores too, as bfloat16 high and low parts (three contraction segments);
    the oracle's P and G are not rounded."""
    worst = run_parity(WL.workload("single"), expect_path=B.PATH_TENSOR)
    assert worst["dw"] <= 1.0 and worst["exempt"] == 0.0
    run_parity(WL.workload("single"), flags=B.FLAG_NO_TENSOR_CORES, expect_path=B.PATH_SIMT)


@pytest.mark.parametrize("rank,shapes", [
    (16, [(64, 72), (72, 64), (128, 128), (16, 520)]),
    (64, [(200, 1000), (1000, 200), (520, 264), (200, 333), (336, 203)]),   # ragged tiles, odd pitches
    (130, [(300, 1032), (1032, 304)]),                                      # rank padded to 144
    (512, [(512, 1376), (1376, 512)]),
])
def test_tensor_core_path_fp32_gradients(rank, shapes):
    wl = _wl(shapes, rank, dtype="f32", steps=4, T=2, wd=0.01)
    worst = run_parity(wl, expect_path=B.PATH_TENSOR)
    assert worst["exempt"] == 0.0
    run_parity(wl, flags=B.FLAG_KEEP_P, expect_path=B.PATH_TENSOR, tuning=B.make_tuning(repitch_mb=1))
    # the ring kernel does not read the split copies: fp32 gradients stay on the CUDA cores there
    opt = B.Apollo(wl.shapes, B.config_for(wl), tuning=B.make_tuning(kernel=B.TC_KERNEL_RING))
    assert opt.path(0) == B.PATH_SIMT
    opt.close()


def test_config_llama60m_mini_all_matrices():
    wl = WL.workload("llama60m_mini")
    run_parity(wl, steps=20, check_mats=[0, 3, 4, 6, 55], expect_path=B.PATH_STREAM)


def test_zero_gradient_and_zero_lr():
    dev = torch.device("cuda")
    shapes = [(33, 130)]
    opt = B.Apollo(shapes, B.make_config(rank=4, dtype=B.DT_F32, flags=B.FLAG_NO_TENSOR_CORES))
    W = torch.randn(33, 130, device=dev) * 0.02
    W0 = W.clone()
    G = torch.zeros_like(W)
    opt.step([W], [G], 0.1, 0.5)
    torch.cuda.synchronize()
    assert torch.all(opt.scales(0) == 0)
    assert torch.allclose(W, W0 * 0.95, rtol=1e-6, atol=0)
    G = torch.randn_like(W) * 1e-3
    W1 = W.clone()
    opt.step([W], [G], 0.0, 0.3)
    torch.cuda.synchronize()
    assert torch.equal(W, W1)
    M, V = opt.state(0)
    assert M.abs().sum() > 0 and V.abs().sum() > 0
    opt.close()


def test_runs_are_bitwise_reproducible():
    wl = _wl([(200, 333), (333, 200)], 8, dtype="bf16", steps=3)
    outs = []
    for _ in range(2):
        opt = B.Apollo(wl.shapes, B.make_config(rank=8, dtype=B.DT_BF16, T=2, seed=9))
        Ws = [WL.make_weight(wl, i).cuda() for i in range(2)]
        for t in range(3):
            opt.step(Ws, [WL.make_grad(wl, i, t).cuda() for i in range(2)], 1e-2, 0.01)
        torch.cuda.synchronize()
        outs.append([w.clone() for w in Ws])
        opt.close()
    assert all(torch.equal(a, b) for a, b in zip(*outs))


def test_misaligned_and_null_pointers_are_rejected_before_any_launch():
    dev = torch.device("cuda")
    opt = B.Apollo([(16, 32)], B.make_config(rank=2, dtype=B.DT_F32))
    buf = torch.zeros(16 * 32 + 4, device=dev)
    W = buf[1:1 + 512].view(16, 32)         # 4-byte offset: not 16-byte aligned
    G = torch.zeros(16, 32, device=dev)
    with pytest.raises(B.ApolloError) as e:
        opt.step([W], [G], 0.1, check=False)
    assert e.value.code == B.ERR_ALIGN
    assert opt.step_count() == 0
    opt.close()


@pytest.mark.parametrize("rank,mode,flags", [(32, "channel", 0), (1, "tensor", 0), (5, "channel", B.FLAG_NO_TENSOR_CORES),
                                             (40, "channel", 0)])      # 40: kept with 48 rows on the tensor path
def test_checkpoint_and_resume_continue_bit_for_bit(rank, mode, flags):
    wl = _wl([(200, 336), (336, 200), (64, 64)], rank, mode=mode, dtype="bf16", T=2, steps=6, wd=0.01)
    dev = torch.device("cuda")
    cfg = B.config_for(wl, flags)

    def run(opt, Ws, t0, t1):
        for t in range(t0, t1):
            opt.step(Ws, [WL.make_grad(wl, i, t).to(dev) for i in range(3)], wl.lr, wl.wd)
        torch.cuda.synchronize()

    whole = B.Apollo(wl.shapes, cfg)
    W_whole = [WL.make_weight(wl, i).to(dev) for i in range(3)]
    run(whole, W_whole, 0, 6)

    first = B.Apollo(wl.shapes, cfg)
    W_part = [WL.make_weight(wl, i).to(dev) for i in range(3)]
    run(first, W_part, 0, 3)                       # stops right after a refresh step (T = 2)
    blob, t = first.state_export(), first.step_count()
    assert t == 3
    first.close()
    second = B.Apollo(wl.shapes, cfg)
    second.state_import(blob.clone(), t)
    run(second, W_part, 3, 6)
    assert second.step_count() == 6
    for a, b in zip(W_whole, W_part):
        assert torch.equal(a, b)
    for i in range(3):
        assert torch.equal(whole.scales(i), second.scales(i))
        assert torch.equal(whole.limiter(i), second.limiter(i))
    fresh = B.Apollo(wl.shapes, cfg)
    with pytest.raises(B.ApolloError):
        fresh.state_export()                       # nothing has run yet


@pytest.mark.parametrize("rank", [32, 40])
@pytest.mark.parametrize("flags", [0, B.FLAG_BF16_STATES])
def test_checkpoint_is_dense_whatever_layout_the_kernels_keep(flags, rank):
    """The tensor path keeps its moments in channel blocks, the CUDA-core path row by row with a padded
    pitch; the checkpoint and apollo_get_state are dense in both, so a state written by one is read by
    the other, entry for entry."""
    shapes = [(200, 336), (336, 203), (64, 64), (128, 520)]     # n = 336, 336, 64, 520: ragged last blocks
    wl = _wl(shapes, rank, dtype="bf16", T=2, steps=3, wd=0.01)
    dev = torch.device("cuda")
    tensor = B.Apollo(wl.shapes, B.config_for(wl, flags))
    assert all(tensor.path(i) == B.PATH_TENSOR for i in range(len(shapes)))
    W = [WL.make_weight(wl, i).to(dev) for i in range(len(shapes))]
    for t in range(3):
        tensor.step(W, [WL.make_grad(wl, i, t).to(dev) for i in range(len(shapes))], wl.lr, wl.wd)
    blob = tensor.state_export()
    cores = B.Apollo(wl.shapes, B.config_for(wl, flags | B.FLAG_NO_TENSOR_CORES))
    assert all(cores.path(i) == B.PATH_SIMT for i in range(len(shapes)))
    cores.state_import(blob.clone(), 3)
    for i in range(len(shapes)):
        (Ma, Va), (Mb, Vb) = tensor.state(i), cores.state(i)
        assert torch.equal(Ma, Mb) and torch.equal(Va, Vb)
        assert Ma.abs().max() > 0 and Va.abs().max() > 0
    assert torch.equal(blob, cores.state_export())
    # and back: a second tensor-path context resumes from the CUDA-core context's checkpoint
    again = B.Apollo(wl.shapes, B.config_for(wl, flags))
    again.state_import(cores.state_export(), 3)
    for i in range(len(shapes)):
        (Ma, Va), (Mb, Vb) = tensor.state(i), again.state(i)
        assert torch.equal(Ma, Mb) and torch.equal(Va, Vb)


@pytest.mark.parametrize("rank,mode,flags,tuning", [
    (32, "channel", 0, {}), (1, "tensor", 0, {}), (5, "channel", B.FLAG_NO_TENSOR_CORES, {}),
    # P generated by the pair kernel's spare warps through a ring of two slots: a range starts in the middle of the ring
    (256, "channel", 0, {"p_generator": 2, "scratch_mb": 1}),
])
def test_layer_wise_range_steps_equal_the_whole_list_step(rank, mode, flags, tuning):
    shapes = [(200, 336), (336, 200), (64, 64), (128, 520), (96, 203), (72, 64), (64, 72)]
    if rank == 256:
        shapes = [(512, 1376), (1376, 512), (512, 512), (300, 1032), (1376, 1400), (520, 264), (264, 520)]
    wl = _wl(shapes, rank, mode=mode, dtype="bf16", T=2, steps=4, wd=0.01)
    dev = torch.device("cuda")
    cfg = B.config_for(wl, flags)
    n = len(shapes)
    whole = B.Apollo(wl.shapes, cfg, tuning=B.make_tuning(**tuning))
    ranged = B.Apollo(wl.shapes, cfg, tuning=B.make_tuning(**tuning))
    Wa = [WL.make_weight(wl, i).to(dev) for i in range(n)]
    Wb = [w.clone() for w in Wa]
    layers = [(4, 7), (2, 4), (0, 2)]          # visited in backward order
    for t in range(4):
        G = [WL.make_grad(wl, i, t).to(dev) for i in range(n)]
        whole.step(Wa, G, wl.lr, wl.wd)
        for k, (a, b) in enumerate(layers):
            ranged.step_range(a, Wb[a:b], G[a:b], wl.lr, wl.wd, close_step=(k == len(layers) - 1))
        torch.cuda.synchronize()
        assert ranged.step_count() == t + 1
        for i in range(n):
            assert torch.equal(Wa[i], Wb[i]), (t, i)
            assert torch.equal(whole.scales(i), ranged.scales(i))
    assert whole.status() == B.OK and ranged.status() == B.OK
    with pytest.raises(B.ApolloError):
        ranged.step_range(5, Wb[5:8] + [Wb[0]], G[5:8] + [G[0]], wl.lr)     # runs past the end of the list


@pytest.mark.parametrize("rank,dtype,flags,path,tuning", [
    (16, "bf16", 0, B.PATH_TENSOR, {}), (4, "f32", 0, B.PATH_SIMT, {}), (6, "bf16", B.FLAG_NO_TENSOR_CORES, B.PATH_SIMT, {}),
    (1, "bf16", 0, B.PATH_STREAM, {}),
    (16, "bf16", 0, B.PATH_TENSOR, {"p_generator": 2}),      # converted by the pair kernel's spare warps
    (16, "bf16", B.FLAG_KEEP_P, B.PATH_TENSOR, {}),
    (24, "f32", 0, B.PATH_TENSOR, {}),                       # fp32 gradients: the supplied P is split into high and low parts
])
def test_caller_supplied_projection_from_an_svd(rank, dtype, flags, path, tuning):
    """The "APOLLO w. SVD" variant: P = top-r left singular vectors of the first gradient (computed here
    with torch on the CPU), handed to the library and to the oracle alike."""
    import numpy as np
    import oracle
    from parity import DW_ABS, DW_REL, SCALE_REL, _f32
    shapes = [(96, 200), (203, 72)]
    wl = _wl(shapes, rank, mode="tensor" if rank == 1 else "channel", dtype=dtype, T=100, steps=3, wd=0.01,
             alpha=1.0)
    dev = torch.device("cuda")
    opt = B.Apollo(wl.shapes, B.config_for(wl, flags), tuning=B.make_tuning(**tuning))
    Ps, orc = [], []
    for i, (rows, cols) in enumerate(shapes):
        assert opt.path(i) == path
        G0 = WL.make_grad(wl, i, 0).float()
        Gv = G0 if rows <= cols else G0.T
        U, _, _ = torch.linalg.svd(Gv.double(), full_matrices=False)
        P = U[:, :rank].T.contiguous().float()              # r x m, orthonormal rows
        if dtype == "bf16" and rank > 1:
            P = P.to(torch.bfloat16).float()                # the operand precision of the projection
        Ps.append(P.to(dev))
        opt.set_projection(i, Ps[-1])
        orc.append(oracle.MatrixOracle(rows, cols, rank=rank, mode=oracle.MODE_TENSOR if rank == 1 else oracle.MODE_CHANNEL,
                                       dtype=oracle.DT_BF16 if dtype == "bf16" else oracle.DT_F32, matrix_id=i,
                                       alpha=1.0, gamma=_f32(wl.gamma), beta1=_f32(wl.beta1), beta2=_f32(wl.beta2),
                                       eps=_f32(wl.eps)))
    W = [WL.make_weight(wl, i).to(dev) for i in range(2)]
    deltas = [torch.zeros(s, dtype=torch.float32, device=dev) for s in shapes]
    opt.set_delta_out(deltas)
    for t in range(3):
        G = [WL.make_grad(wl, i, t) for i in range(2)]
        Wc = [w.float().cpu().numpy() for w in W]
        opt.step(W, [g.to(dev) for g in G], wl.lr, wl.wd)
        torch.cuda.synchronize()
        for i in range(2):
            res = orc[i].step(Wc[i], G[i].float().numpy(), _f32(wl.lr), _f32(wl.wd), P=Ps[i].double().cpu().numpy())
            bound = DW_REL * np.max(np.abs(res.dW)) + DW_ABS
            assert np.max(np.abs(deltas[i].cpu().numpy() - res.dW)) <= bound
            s_gpu = opt.scales(i).cpu().numpy()
            assert np.max(np.abs(s_gpu - res.s) / np.abs(res.s)) <= SCALE_REL
            W[i].copy_(torch.from_numpy(res.W).to(W[i].dtype))
    opt.set_projection(0, None)                             # back to the generator
    opt.close()


@pytest.mark.parametrize("rank,mode,flags,shapes", [
    (64, "channel", B.FLAG_BF16_STATES, [(200, 1000), (1000, 200), (520, 264)]),
    (256, "channel", B.FLAG_BF16_STATES, [(512, 1376), (1376, 512)]),
    (5, "channel", B.FLAG_BF16_STATES | B.FLAG_NO_TENSOR_CORES, [(33, 130), (130, 33)]),
    (1, "tensor", B.FLAG_BF16_STATES, [(600, 2600), (3000, 2100)]),
])
def test_bf16_moment_storage(rank, mode, flags, shapes):
    wl = _wl(shapes, rank, mode=mode, dtype="bf16", steps=5, T=2, wd=0.01,
             alpha=math.sqrt(128.0) if mode == "tensor" else 1.0)
    run_parity(wl, flags=flags)
    # the workspace shrinks by two bytes per moment entry
    full = B.workspace_bytes(shapes, B.config_for(wl, flags & ~B.FLAG_BF16_STATES))
    half = B.workspace_bytes(shapes, B.config_for(wl, flags))
    moments = sum(2 * rank * max(s) for s in shapes)
    assert full - half >= 2 * moments - 4096 * len(shapes)
    # state read-back is widened to float and holds bfloat16 values
    opt = B.Apollo(shapes, B.config_for(wl, flags))
    W = [WL.make_weight(wl, i).cuda() for i in range(len(shapes))]
    opt.step(W, [WL.make_grad(wl, i, 0).cuda() for i in range(len(shapes))], 1e-2)
    M, V = opt.state(0)
    assert torch.equal(M, M.to(torch.bfloat16).float()) and torch.equal(V, V.to(torch.bfloat16).float())
    blob = opt.state_export()
    assert blob.numel() == sum(2 * 2 * rank * max(s) + 4 for s in shapes)
    opt.close()


def test_a_wait_that_runs_out_is_reported_and_leaves_the_context_usable():
    """Every wait of the tensor kernel is bounded; the self-test kernel lets one run out on purpose
    (an mbarrier nothing arrives on).  The status word turns into ERR_TIMEOUT once, and the optimizer
    goes on exactly as a context that never saw it."""
    wl = _wl([(256, 520), (520, 256)], 32, dtype="bf16", steps=3, T=2)
    dev = torch.device("cuda")
    a, b = B.Apollo(wl.shapes, B.config_for(wl)), B.Apollo(wl.shapes, B.config_for(wl))
    with pytest.raises(B.ApolloError):
        a.selftest_bounded_wait()                 # no step yet: no status word
    Wa = [WL.make_weight(wl, i).to(dev) for i in range(2)]
    Wb = [w.clone() for w in Wa]
    for t in range(3):
        G = [WL.make_grad(wl, i, t).to(dev) for i in range(2)]
        a.step(Wa, G, wl.lr, wl.wd)
        b.step(Wb, G, wl.lr, wl.wd)
        if t == 0:
            assert a.status() == B.OK
            a.selftest_bounded_wait()
            assert a.status() == B.ERR_TIMEOUT     # reported once ...
            assert a.status() == B.OK              # ... and cleared
    assert a.status() == B.OK and b.status() == B.OK
    for x, y in zip(Wa, Wb):
        assert torch.equal(x, y)


def test_a_step_whose_projection_gave_up_leaves_weights_and_limiter_untouched():
    """Once the status word says that a wait has run out, the finalize and update passes of a step write
    nothing: the weights and the limiter's norm stay as they were until the caller has read the status."""
    wl = _wl([(512, 1376), (1376, 512)], 64, dtype="bf16", steps=3, T=2, wd=0.01)
    dev = torch.device("cuda")
    opt = B.Apollo(wl.shapes, B.config_for(wl))
    W = [WL.make_weight(wl, i).to(dev) for i in range(2)]
    opt.step(W, [WL.make_grad(wl, i, 0).to(dev) for i in range(2)], wl.lr, wl.wd)
    assert opt.status() == B.OK
    W_before = [w.clone() for w in W]
    lim_before = [opt.limiter(i).clone() for i in range(2)]
    opt.selftest_bounded_wait()                   # the status word now reads "timeout", as after a wait that gave up
    opt.step(W, [WL.make_grad(wl, i, 1).to(dev) for i in range(2)], wl.lr, wl.wd)
    torch.cuda.synchronize()
    for a, b in zip(W, W_before):
        assert torch.equal(a, b)
    for i in range(2):
        assert torch.equal(opt.limiter(i), lim_before[i])
    assert opt.status() == B.ERR_TIMEOUT
    assert opt.status() == B.OK
    opt.step(W, [WL.make_grad(wl, i, 2).to(dev) for i in range(2)], wl.lr, wl.wd)     # the context works on
    torch.cuda.synchronize()
    assert opt.status() == B.OK
    assert not torch.equal(W[0], W_before[0])
    opt.close()

