"""Host-side checks of the C-ABI library that need no GPU: every declared symbol is
exported, and workspace planning validates shapes and configuration."""
import re
from pathlib import Path

import pytest

from paper_2412_05270_b200 import binding as B
from paper_2412_05270_b200.build import build_library

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()


def test_library_exports_every_declared_symbol():
    header = (ROOT / "include" / "apollo.h").read_text()
    declared = set(re.findall(r"\b(apollo_[a-z_0-9]+)\s*\(", header))
    declared -= {"apollo_ctx", "apollo_shape", "apollo_config"}
    lib = B.load()
    assert declared == set(B.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name
    # the bounds-checking build is the same library with checks compiled in
    from paper_2412_05270_b200.build import build_library
    import ctypes
    debug = ctypes.CDLL(str(build_library(debug=True)))
    for name in declared:
        assert hasattr(debug, name), name


def test_strerror_names_every_code():
    for code in range(0, -11, -1):
        assert B.strerror(code) and "unknown" not in B.strerror(code)
    assert "unknown" in B.strerror(-99)


def test_tuning_is_validated_and_sizes_the_p_scratch():
    shapes = [(4096, 4096)] * 100
    cfg = B.make_config(rank=256, dtype=B.DT_BF16)
    moments = 100 * 2 * 256 * 4096 * 4
    per_step = B.workspace_bytes(shapes, cfg)
    kept = B.workspace_bytes(shapes, B.make_config(rank=256, dtype=B.DT_BF16, flags=B.FLAG_KEEP_P))
    p_bytes = 256 * 4096 * 2
    # 200 MB of projections do not fit the 128 MB scratch: a ring of 32 MB (16 slots of 2 MB); kept: one slot per matrix
    assert per_step - moments < 56 << 20       # ring + scales, partial sums, tables
    assert kept - per_step == (100 - 16) * p_bytes
    assert B.workspace_bytes(shapes, cfg, B.make_tuning(scratch_mb=8)) == per_step - (16 - 4) * p_bytes
    # 80 MB of projections fit: all of them are regenerated into the scratch by the generator kernel every step
    few = [(4096, 4096)] * 40
    assert B.workspace_bytes(few, B.make_config(rank=256, dtype=B.DT_BF16, flags=B.FLAG_KEEP_P)) == B.workspace_bytes(few, cfg)
    for bad in (dict(kernel=2), dict(p_source=3), dict(r_slice=24), dict(r_slice=512), dict(nblk=3),
                dict(nblk=4, r_slice=256), dict(scratch_mb=-1), dict(epi_prefetch=9), dict(p_generator=3), dict(realign=3), dict(repitch_mb=-1)):
        with pytest.raises(B.ApolloError) as err:
            B.workspace_bytes(shapes, cfg, B.make_tuning(**bad))
        assert err.value.code == B.ERR_INVALID_ARG, bad


def test_workspace_grows_with_rank_and_counts_moments():
    shapes = [(512, 1376), (1376, 512)]
    small = B.workspace_bytes(shapes, B.make_config(rank=16, dtype=B.DT_BF16))
    big = B.workspace_bytes(shapes, B.make_config(rank=128, dtype=B.DT_BF16))
    moments_small = 2 * 2 * 16 * 1376 * 4
    moments_big = 2 * 2 * 128 * 1376 * 4
    assert small >= moments_small and big >= moments_big
    assert big - small >= (moments_big - moments_small)
    mini = B.workspace_bytes(shapes, B.make_config(rank=1, mode=B.SCALE_TENSOR))
    assert mini < small


@pytest.mark.parametrize("shapes,kw,code", [
    ([(4, 9)], dict(rank=5), B.ERR_RANK),
    ([(4, 9)], dict(rank=0), B.ERR_RANK),
    ([(1024, 1024)], dict(rank=513), B.ERR_RANK),
    ([(0, 9)], dict(rank=1), B.ERR_SHAPE),
    ([(4, 2**31)], dict(rank=1), B.ERR_SHAPE),
    ([(4, 9)], dict(rank=1, T=0), B.ERR_INVALID_ARG),
    ([(4, 9)], dict(rank=1, mode=2), B.ERR_INVALID_ARG),
    ([(4, 9)], dict(rank=1, dtype=3), B.ERR_INVALID_ARG),
    ([(4, 9)], dict(rank=1, beta1=1.5), B.ERR_INVALID_ARG),
    ([(4, 9)], dict(rank=1, eps=float("nan")), B.ERR_INVALID_ARG),
    ([(4, 9)], dict(rank=1, beta2=1.0, bias_correction=True), B.ERR_INVALID_ARG),
    ([], dict(rank=1), B.ERR_INVALID_ARG),
])
def test_invalid_arguments_are_rejected(shapes, kw, code):
    with pytest.raises(B.ApolloError) as e:
        B.workspace_bytes(shapes, B.make_config(**kw))
    assert e.value.code == code


def test_square_and_rank_equal_to_short_side_are_accepted():
    assert B.workspace_bytes([(6, 6)], B.make_config(rank=6)) > 0
    assert B.workspace_bytes([(3, 1)], B.make_config(rank=1)) > 0
