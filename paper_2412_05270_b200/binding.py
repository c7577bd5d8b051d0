"""ctypes binding of libapollo.so: argument marshalling only.

Every step of the optimizer runs inside the library's CUDA kernels; PyTorch supplies device
memory and the stream.  There is no CPU fallback: if the shared library is missing the
import of this module's symbols raises.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libapollo.so"
DEBUG_LIB_PATH = _PKG / "libapollo_debug.so"     # built with -DAPOLLO_DEBUG: index checks inside every kernel

OK = 0
ERR_INVALID_ARG, ERR_SHAPE, ERR_RANK, ERR_ALIGN, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_UNSUPPORTED = (
    -1, -2, -3, -4, -5, -6, -7, -8)
ERR_TOO_LARGE = -9
ERR_INTERNAL = -10
STATIC_SCRATCH_BYTES = 8 << 20
SCALE_CHANNEL, SCALE_TENSOR = 0, 1
DT_F32, DT_BF16 = 0, 1
FLAG_NO_TENSOR_CORES = 1
FLAG_BF16_STATES = 2
FLAG_KEEP_P = 4
TC_KERNEL_PAIR, TC_KERNEL_RING = 0, 1
P_SCRATCH, P_SHARED = 0, 1
PATH_STREAM, PATH_SIMT, PATH_TENSOR = 0, 1, 2

EXPORTS = [
    "apollo_workspace_bytes", "apollo_create", "apollo_step", "apollo_destroy", "apollo_step_count",
    "apollo_get_scales", "apollo_get_limiter", "apollo_get_state", "apollo_set_delta_out", "apollo_status",
    "apollo_philox_draws", "apollo_projection", "apollo_get_path", "apollo_last_launches", "apollo_strerror",
    "apollo_set_timing", "apollo_get_timing", "apollo_mini_step_static", "apollo_cuda_error_string", "apollo_adamw_step",
    "apollo_state_bytes", "apollo_state_export", "apollo_state_import", "apollo_step_range", "apollo_set_projection",
    "apollo_selftest_bounded_wait", "apollo_workspace_bytes_tuned", "apollo_create_tuned",
]


class ApolloError(RuntimeError):
    def __init__(self, code: int, what: str):
        detail = f" [{load().apollo_cuda_error_string().decode()}]" if code == ERR_CUDA else ""
        super().__init__(f"{what}: {strerror(code)} ({code}){detail}")
        self.code = code


class Shape(ctypes.Structure):
    _fields_ = [("rows", ctypes.c_int64), ("cols", ctypes.c_int64)]


class Config(ctypes.Structure):
    _fields_ = [
        ("rank", ctypes.c_int32), ("mode", ctypes.c_int32), ("dtype", ctypes.c_int32), ("T", ctypes.c_int32),
        ("seed", ctypes.c_uint64),
        ("alpha", ctypes.c_float), ("gamma", ctypes.c_float),
        ("beta1", ctypes.c_float), ("beta2", ctypes.c_float), ("eps", ctypes.c_float),
        ("bias_correction", ctypes.c_int32), ("flags", ctypes.c_uint32),
    ]


class Tuning(ctypes.Structure):
    """apollo_tuning: zero fields select the defaults."""
    _fields_ = [("kernel", ctypes.c_int32), ("p_source", ctypes.c_int32), ("p_generator", ctypes.c_int32),
                ("scratch_mb", ctypes.c_int32), ("r_slice", ctypes.c_int32), ("nblk", ctypes.c_int32),
                ("epi_prefetch", ctypes.c_int32), ("realign", ctypes.c_int32), ("repitch_mb", ctypes.c_int32)]


def make_tuning(kernel=TC_KERNEL_PAIR, p_source=P_SCRATCH, p_generator=0, scratch_mb=0, r_slice=0, nblk=0,
                epi_prefetch=None, realign=0, repitch_mb=0) -> Tuning:
    """epi_prefetch: distance in chunks (0 = no prefetch), None = the default."""
    return Tuning(int(kernel), int(p_source), int(p_generator), int(scratch_mb), int(r_slice), int(nblk),
                  0 if epi_prefetch is None else int(epi_prefetch) + 1, int(realign), int(repitch_mb))


_lib = None


_libs = {}


def use_library(path=None):
    """Route all later calls of this module through the library at `path` (None: libapollo.so); the test of
    the bounds-checking build switches to libapollo_debug.so and back.  Contexts keep the library they were
    created with."""
    global _lib
    _lib = None if path is None else _load_from(Path(path))


def load():
    """Load libapollo.so; raises if it has not been built (there is no fallback)."""
    global _lib
    if _lib is None:
        _lib = _load_from(LIB_PATH)
    return _lib


def _load_from(path: Path):
    if path in _libs:
        return _libs[path]
    if not path.exists():
        raise ImportError(f"{path} is missing: run `python -m paper_2412_05270_b200.build` (nvcc, sm_100a)")
    lib = ctypes.CDLL(str(path))
    vp, i32, u32, u64, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_uint32, ctypes.c_uint64, ctypes.c_float
    lib.apollo_workspace_bytes.argtypes = [ctypes.POINTER(Shape), i32, ctypes.POINTER(Config),
                                           ctypes.POINTER(ctypes.c_size_t)]
    lib.apollo_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(Shape), i32, ctypes.POINTER(Config), vp,
                                  ctypes.c_size_t]
    lib.apollo_workspace_bytes_tuned.argtypes = [ctypes.POINTER(Shape), i32, ctypes.POINTER(Config),
                                                 ctypes.POINTER(Tuning), ctypes.POINTER(ctypes.c_size_t)]
    lib.apollo_create_tuned.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(Shape), i32, ctypes.POINTER(Config),
                                        ctypes.POINTER(Tuning), vp, ctypes.c_size_t]
    lib.apollo_step.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(vp), f32, f32, vp]
    lib.apollo_step_range.argtypes = [vp, i32, i32, ctypes.POINTER(vp), ctypes.POINTER(vp), f32, f32, i32, vp]
    lib.apollo_set_projection.argtypes = [vp, i32, vp]
    lib.apollo_destroy.argtypes = [vp]
    lib.apollo_step_count.argtypes = [vp, ctypes.POINTER(ctypes.c_int64)]
    lib.apollo_get_scales.argtypes = [vp, i32, vp, vp]
    lib.apollo_get_limiter.argtypes = [vp, i32, vp, vp]
    lib.apollo_get_state.argtypes = [vp, i32, vp, vp, vp]
    lib.apollo_set_delta_out.argtypes = [vp, ctypes.POINTER(vp)]
    lib.apollo_status.argtypes = [vp, vp]
    lib.apollo_selftest_bounded_wait.argtypes = [vp, vp]
    lib.apollo_philox_draws.argtypes = [u64, u32, u32, i32, i32, vp, vp]
    lib.apollo_projection.argtypes = [u64, u32, u32, i32, i32, vp, vp]
    lib.apollo_get_path.argtypes = [vp, i32, ctypes.POINTER(i32)]
    lib.apollo_last_launches.argtypes = [vp, ctypes.POINTER(i32)]
    lib.apollo_set_timing.argtypes = [vp, i32]
    lib.apollo_get_timing.argtypes = [vp, i32, ctypes.POINTER(f32)]
    lib.apollo_mini_step_static.argtypes = [vp, vp, ctypes.c_int64, ctypes.c_int64, vp, vp, vp,
                                            ctypes.POINTER(Config), u32, ctypes.c_int64, f32, f32, vp]
    lib.apollo_strerror.argtypes = [ctypes.c_int]
    lib.apollo_strerror.restype = ctypes.c_char_p
    lib.apollo_adamw_step.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(vp),
                                      ctypes.POINTER(ctypes.c_int64), i32, i32, f32, f32, f32, f32, f32,
                                      ctypes.c_int64, i32, ctypes.POINTER(vp), vp]
    lib.apollo_state_bytes.argtypes = [vp, ctypes.POINTER(ctypes.c_size_t)]
    lib.apollo_state_export.argtypes = [vp, vp, vp]
    lib.apollo_state_import.argtypes = [vp, vp, ctypes.c_int64, vp]
    lib.apollo_cuda_error_string.argtypes = []
    lib.apollo_cuda_error_string.restype = ctypes.c_char_p
    for name in EXPORTS:
        if name not in ("apollo_strerror", "apollo_cuda_error_string"):
            getattr(lib, name).restype = ctypes.c_int
    _libs[path] = lib
    return lib


def strerror(code: int) -> str:
    return load().apollo_strerror(code).decode()


def _check(code: int, what: str):
    if code != OK:
        raise ApolloError(code, what)


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream


def _shape_array(shapes):
    arr = (Shape * len(shapes))()
    for i, (r, c) in enumerate(shapes):
        arr[i].rows, arr[i].cols = int(r), int(c)
    return arr


def make_config(rank, mode=SCALE_CHANNEL, dtype=DT_BF16, T=200, seed=0, alpha=1.0, gamma=1.01,
                beta1=0.9, beta2=0.999, eps=1e-8, bias_correction=False, flags=0) -> Config:
    return Config(int(rank), int(mode), int(dtype), int(T), int(seed), float(alpha), float(gamma),
                  float(beta1), float(beta2), float(eps), int(bool(bias_correction)), int(flags))


def config_for(wl, flags=0, bias_correction=False) -> Config:
    """The library configuration of a named workload (see workloads.py)."""
    return make_config(rank=wl.rank, mode=SCALE_TENSOR if wl.mode == "tensor" else SCALE_CHANNEL,
                       dtype=DT_BF16 if wl.dtype == "bf16" else DT_F32, T=wl.T, seed=wl.seed,
                       alpha=wl.alpha, gamma=wl.gamma, beta1=wl.beta1, beta2=wl.beta2, eps=wl.eps,
                       bias_correction=bias_correction, flags=flags)


def workspace_bytes(shapes, cfg: Config, tuning: Tuning | None = None) -> int:
    out = ctypes.c_size_t(0)
    if tuning is None:
        _check(load().apollo_workspace_bytes(_shape_array(shapes), len(shapes), ctypes.byref(cfg), ctypes.byref(out)),
               "apollo_workspace_bytes")
    else:
        _check(load().apollo_workspace_bytes_tuned(_shape_array(shapes), len(shapes), ctypes.byref(cfg),
                                                   ctypes.byref(tuning), ctypes.byref(out)),
               "apollo_workspace_bytes_tuned")
    return out.value


def philox_draws(seed: int, matrix: int, epoch: int, r: int, m: int, stream=None) -> torch.Tensor:
    out = torch.empty((r, (m + 3) // 4, 4), dtype=torch.int32, device="cuda")
    _check(load().apollo_philox_draws(seed, matrix, epoch, r, m, out.data_ptr(), _stream_ptr(stream)),
           "apollo_philox_draws")
    return out


def projection(seed: int, matrix: int, epoch: int, r: int, m: int, stream=None) -> torch.Tensor:
    out = torch.empty((r, m), dtype=torch.float32, device="cuda")
    _check(load().apollo_projection(seed, matrix, epoch, r, m, out.data_ptr(), _stream_ptr(stream)),
           "apollo_projection")
    return out


def mini_step_static(W, G, M, V, prev_norm, cfg: Config, matrix: int, t: int, lr: float, wd: float = 0.0,
                     stream=None):
    """apollo_mini_step_static: a rank-1 step for one matrix that allocates nothing.

    For callers that cannot get device memory when the optimizer has to run (see the
    header): W, G are the weight and gradient, M, V (n floats) and prev_norm (1 float) the
    state the caller keeps between steps; the temporaries live in a fixed array inside the
    library, shared by all calls on the device, so calls must not overlap on the GPU.
    """
    rows, cols = W.shape
    _check(load().apollo_mini_step_static(W.data_ptr(), G.data_ptr(), rows, cols, M.data_ptr(), V.data_ptr(),
                                          prev_norm.data_ptr(), ctypes.byref(cfg), matrix, t, lr, wd,
                                          _stream_ptr(stream)), "apollo_mini_step_static")


def adamw_step(params, grads, ms, vs, t, lr, beta1=0.9, beta2=0.999, eps=1e-8, wd=0.0, bias_correction=True,
               deltas=None, stream=None):
    """apollo_adamw_step over lists of CUDA tensors (params/grads of one dtype; ms/vs fp32, same numel)."""
    n = len(params)
    dtype = DT_BF16 if params[0].dtype == torch.bfloat16 else DT_F32

    def arr(ts):
        a = (ctypes.c_void_p * n)()
        for i, x in enumerate(ts):
            a[i] = None if x is None else x.data_ptr()
        return a
    numel = (ctypes.c_int64 * n)(*[p.numel() for p in params])
    _check(load().apollo_adamw_step(arr(params), arr(grads), arr(ms), arr(vs), numel, n, dtype, lr, beta1, beta2, eps,
                                    wd, t, int(bool(bias_correction)), arr(deltas) if deltas is not None else None,
                                    _stream_ptr(stream)), "apollo_adamw_step")


class Apollo:
    """apollo_create / apollo_step over a list of CUDA tensors (same dtype, 2-D, contiguous)."""

    def __init__(self, shapes, cfg: Config, device="cuda", tuning: Tuning | None = None):
        self.lib = load()
        self.shapes = [(int(r), int(c)) for r, c in shapes]
        self.cfg = cfg
        self.device = torch.device(device)
        nbytes = workspace_bytes(self.shapes, cfg, tuning)
        self.workspace_bytes = nbytes
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
            base = self.workspace.data_ptr()
            self._ws_ptr = (base + 255) // 256 * 256
            ctx = ctypes.c_void_p()
            if tuning is None:
                _check(self.lib.apollo_create(ctypes.byref(ctx), _shape_array(self.shapes), len(self.shapes),
                                              ctypes.byref(cfg), self._ws_ptr, nbytes), "apollo_create")
            else:
                _check(self.lib.apollo_create_tuned(ctypes.byref(ctx), _shape_array(self.shapes), len(self.shapes),
                                                    ctypes.byref(cfg), ctypes.byref(tuning), self._ws_ptr, nbytes),
                       "apollo_create_tuned")
        self.ctx = ctx
        self._delta = None
        self._w_arr = (ctypes.c_void_p * len(self.shapes))()
        self._g_arr = (ctypes.c_void_p * len(self.shapes))()

    def close(self):
        if getattr(self, "ctx", None):
            self.lib.apollo_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check_tensors(self, Ws, Gs):
        want = torch.bfloat16 if self.cfg.dtype == DT_BF16 else torch.float32
        if len(Ws) != len(self.shapes) or len(Gs) != len(self.shapes):
            raise ValueError("parameter list length differs from the context's")
        for w, g, shp in zip(Ws, Gs, self.shapes):
            for x in (w, g):
                if not x.is_cuda or x.dtype != want or tuple(x.shape) != shp or not x.is_contiguous():
                    raise ValueError("tensors must be contiguous CUDA tensors of the context's dtype and shapes")

    def step(self, Ws, Gs, lr: float, wd: float = 0.0, stream=None, check: bool = True):
        if check:
            self._check_tensors(Ws, Gs)
        for i, (w, g) in enumerate(zip(Ws, Gs)):
            self._w_arr[i] = w.data_ptr()
            self._g_arr[i] = g.data_ptr()
        _check(self.lib.apollo_step(self.ctx, self._w_arr, self._g_arr, lr, wd, _stream_ptr(stream)), "apollo_step")

    def step_range(self, first: int, Ws, Gs, lr: float, wd: float = 0.0, close_step: bool = False, stream=None):
        """apollo_step_range: the step of matrices first .. first + len(Ws) - 1 (layer-wise updates)."""
        n = len(Ws)
        w = (ctypes.c_void_p * n)(*[x.data_ptr() for x in Ws])
        g = (ctypes.c_void_p * n)(*[x.data_ptr() for x in Gs])
        _check(self.lib.apollo_step_range(self.ctx, first, n, w, g, lr, wd, int(close_step), _stream_ptr(stream)),
               "apollo_step_range")

    def set_projection(self, mat: int, P):
        """Use the fp32 CUDA tensor P (r x m) as the projection of matrix `mat`; None restores the generator."""
        if P is not None:
            m = min(self.shapes[mat])
            assert P.is_cuda and P.dtype == torch.float32 and tuple(P.shape) == (self.cfg.rank, m) and P.is_contiguous()
            self._ext_p = getattr(self, "_ext_p", {})
            self._ext_p[mat] = P                      # keep it alive
        _check(self.lib.apollo_set_projection(self.ctx, mat, None if P is None else P.data_ptr()),
               "apollo_set_projection")

    def set_delta_out(self, deltas):
        """deltas: list of float32 CUDA tensors shaped like the weights (None entries skip a matrix), or None."""
        if deltas is None:
            _check(self.lib.apollo_set_delta_out(self.ctx, None), "apollo_set_delta_out")
            self._delta = None
            return
        arr = (ctypes.c_void_p * len(self.shapes))()
        for i, d in enumerate(deltas):
            if d is None:
                arr[i] = None
                continue
            assert d.is_cuda and d.dtype == torch.float32 and tuple(d.shape) == self.shapes[i] and d.is_contiguous()
            arr[i] = d.data_ptr()
        _check(self.lib.apollo_set_delta_out(self.ctx, arr), "apollo_set_delta_out")
        self._delta = deltas

    def scales(self, mat: int, stream=None) -> torch.Tensor:
        out = torch.empty(max(self.shapes[mat]), dtype=torch.float32, device=self.device)
        _check(self.lib.apollo_get_scales(self.ctx, mat, out.data_ptr(), _stream_ptr(stream)), "apollo_get_scales")
        return out

    def limiter(self, mat: int, stream=None) -> torch.Tensor:
        out = torch.empty(4, dtype=torch.float32, device=self.device)
        _check(self.lib.apollo_get_limiter(self.ctx, mat, out.data_ptr(), _stream_ptr(stream)), "apollo_get_limiter")
        return out

    def state(self, mat: int, stream=None):
        n = max(self.shapes[mat])
        M = torch.empty((self.cfg.rank, n), dtype=torch.float32, device=self.device)
        V = torch.empty_like(M)
        _check(self.lib.apollo_get_state(self.ctx, mat, M.data_ptr(), V.data_ptr(), _stream_ptr(stream)),
               "apollo_get_state")
        return M, V

    def status(self, stream=None) -> int:
        return self.lib.apollo_status(self.ctx, _stream_ptr(stream))

    def selftest_bounded_wait(self, stream=None):
        """Launches the kernel whose only wait runs out; the next status() then reports ERR_TIMEOUT."""
        _check(self.lib.apollo_selftest_bounded_wait(self.ctx, _stream_ptr(stream)), "apollo_selftest_bounded_wait")

    def path(self, mat: int) -> int:
        out = ctypes.c_int32(-1)
        _check(self.lib.apollo_get_path(self.ctx, mat, ctypes.byref(out)), "apollo_get_path")
        return out.value

    def step_count(self) -> int:
        out = ctypes.c_int64(0)
        _check(self.lib.apollo_step_count(self.ctx, ctypes.byref(out)), "apollo_step_count")
        return out.value

    def state_export(self, stream=None) -> torch.Tensor:
        """The optimizer state (moments and limiter norms) as one flat uint8 CUDA tensor."""
        n = ctypes.c_size_t(0)
        _check(self.lib.apollo_state_bytes(self.ctx, ctypes.byref(n)), "apollo_state_bytes")
        out = torch.empty(n.value, dtype=torch.uint8, device=self.device)
        _check(self.lib.apollo_state_export(self.ctx, out.data_ptr(), _stream_ptr(stream)), "apollo_state_export")
        return out

    def state_import(self, flat: torch.Tensor, step_count: int, stream=None):
        n = ctypes.c_size_t(0)
        _check(self.lib.apollo_state_bytes(self.ctx, ctypes.byref(n)), "apollo_state_bytes")
        assert flat.is_cuda and flat.dtype == torch.uint8 and flat.numel() == n.value and flat.is_contiguous()
        _check(self.lib.apollo_state_import(self.ctx, flat.data_ptr(), step_count, _stream_ptr(stream)),
               "apollo_state_import")

    def set_timing(self, on: bool):
        _check(self.lib.apollo_set_timing(self.ctx, int(on)), "apollo_set_timing")

    def timing(self, steps_back: int = 0):
        """{projection, finalize, update, whole step} of a recent step, in milliseconds."""
        out = (ctypes.c_float * 4)()
        _check(self.lib.apollo_get_timing(self.ctx, steps_back, out), "apollo_get_timing")
        return list(out)

    def last_launches(self) -> int:
        out = ctypes.c_int32(0)
        _check(self.lib.apollo_last_launches(self.ctx, ctypes.byref(out)), "apollo_last_launches")
        return out.value
