"""ctypes binding of ``libmamba_spec.so``: argument marshalling only.

The functions carry the C names (``mamba_spec_init`` / ``mamba_spec_verify`` /
``mamba_spec_commit`` ...) and pass raw device pointers of torch tensors; every
step of the verification call runs in the library's CUDA kernels.  There is no
fallback of any kind: if the shared library is missing, importing this module
raises.  ``Verifier`` is a small convenience wrapper that keeps a context and
checks tensor dtypes/shapes before handing pointers over.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

_LIB_PATH = Path(__file__).resolve().parent / "libmamba_spec.so"
if not _LIB_PATH.exists():
    raise ImportError(
        f"{_LIB_PATH} is missing: build it with `python -m paper_2408_15237_b200.build` "
        "(needs nvcc).  This package has no CPU or PyTorch fallback.")
lib = ctypes.CDLL(str(_LIB_PATH))

OK = 0
DTYPE_F32, DTYPE_BF16 = 0, 1
FLAG_GATE, FLAG_CONV_SILU, FLAG_Y_F32, FLAG_STATE_K = 1, 2, 4, 8
FLAG_MAMBA1, FLAG_DT_SOFTPLUS, FLAG_COMMIT_SELECTS, FLAG_GATED_RMSNORM, FLAG_CONV_BC = 16, 32, 64, 128, 256
STATUS_NPREV_CLAMPED, STATUS_ACCEPT_CLAMPED, STATUS_COPY_TIMEOUT = 1, 2, 4
KERNEL_AUTO, KERNEL_GENERIC, KERNEL_STREAM = 0, 1, 2
ERR_INVALID_ARG, ERR_BAD_SHAPE, ERR_MISALIGNED, ERR_UNSUPPORTED, ERR_CUDA, ERR_NOT_INIT = -1, -2, -3, -4, -5, -6


class Config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "batch_max", "n_layers", "n_heads", "head_dim", "d_state", "n_groups_b", "n_groups_c", "conv_width",
        "k_max", "act_dtype", "flags", "device", "kernel_select")]


class IO(ctypes.Structure):
    _fields_ = [("conv_w", ctypes.c_void_p), ("conv_b", ctypes.c_void_p), ("z", ctypes.c_void_p),
                ("y", ctypes.c_void_p), ("batch", ctypes.c_int32), ("layer", ctypes.c_int32),
                ("t_max", ctypes.c_int32), ("stream", ctypes.c_void_p), ("state_k", ctypes.c_void_p),
                ("conv_state_k", ctypes.c_void_p), ("dt_bias", ctypes.c_void_p), ("norm_weight", ctypes.c_void_p),
                ("norm_eps", ctypes.c_float), ("conv_state_bc", ctypes.c_void_p), ("conv_w_bc", ctypes.c_void_p),
                ("conv_b_bc", ctypes.c_void_p)]


_vp, _i32 = ctypes.c_void_p, ctypes.c_int32
lib.mamba_spec_init.restype = ctypes.c_int
lib.mamba_spec_init.argtypes = [ctypes.POINTER(Config), ctypes.POINTER(_vp)]
lib.mamba_spec_verify.restype = ctypes.c_int
lib.mamba_spec_verify.argtypes = [_vp] * 10 + [_i32, ctypes.POINTER(IO)]
lib.mamba_spec_verify_new.restype = ctypes.c_int
lib.mamba_spec_verify_new.argtypes = [_vp] * 9 + [_i32, ctypes.POINTER(IO)]
lib.mamba_spec_verify_host.restype = ctypes.c_int
lib.mamba_spec_verify_host.argtypes = [_vp] * 10 + [_i32, ctypes.POINTER(IO)]
lib.mamba_spec_verify_host_static.restype = ctypes.c_int
lib.mamba_spec_verify_host_static.argtypes = [ctypes.POINTER(Config)] + [_vp] * 9 + [_i32, ctypes.POINTER(IO), _vp]
lib.mamba_spec_commit.restype = ctypes.c_int
lib.mamba_spec_commit.argtypes = [_vp, _vp, _i32, _vp]
lib.mamba_spec_status.restype = ctypes.c_int
lib.mamba_spec_status.argtypes = [_vp, ctypes.POINTER(_i32)]
lib.mamba_spec_get_n_prev.restype = ctypes.c_int
lib.mamba_spec_get_n_prev.argtypes = [_vp, ctypes.POINTER(_i32), _i32]
lib.mamba_spec_get_selection.restype = ctypes.c_int
lib.mamba_spec_get_selection.argtypes = [_vp, ctypes.POINTER(_i32), _i32]
lib.mamba_spec_describe_plan.restype = ctypes.c_int
lib.mamba_spec_describe_plan.argtypes = [ctypes.POINTER(Config), _i32, _i32, _i32, _i32, ctypes.c_int64, ctypes.c_char_p, _i32]
lib.mamba_spec_launch_count.restype = ctypes.c_int64
lib.mamba_spec_launch_count.argtypes = [_vp]
lib.mamba_spec_last_kernel.restype = ctypes.c_char_p
lib.mamba_spec_last_kernel.argtypes = [_vp]
lib.mamba_spec_last_error.restype = ctypes.c_char_p
lib.mamba_spec_last_error.argtypes = [_vp]
lib.mamba_spec_destroy.restype = None
lib.mamba_spec_destroy.argtypes = [_vp]


class MambaSpecError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"mamba_spec error {code}: {msg}")
        self.code = code


def _ptr(t) -> int | None:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def mamba_spec_init(cfg: Config) -> int:
    """Returns the opaque context handle (an int) or raises MambaSpecError."""
    out = _vp()
    rc = lib.mamba_spec_init(ctypes.byref(cfg), ctypes.byref(out))
    if rc != OK:
        raise MambaSpecError(rc, lib.mamba_spec_last_error(None).decode())
    return out.value


def _check(ctx, rc):
    if rc != OK:
        raise MambaSpecError(rc, lib.mamba_spec_last_error(ctx).decode())


def mamba_spec_verify(ctx, state, conv_state, x, dt, B, C, A, D, n_prev_accepted, k_draft, io: IO) -> None:
    _check(ctx, lib.mamba_spec_verify(ctx, _ptr(state), _ptr(conv_state), _ptr(x), _ptr(dt), _ptr(B), _ptr(C),
                                      _ptr(A), _ptr(D), _ptr(n_prev_accepted), int(k_draft), ctypes.byref(io)))


def mamba_spec_verify_new(ctx, state, conv_state, x_new, dt_new, B_new, C_new, A, D, k_draft, io: IO) -> None:
    _check(ctx, lib.mamba_spec_verify_new(ctx, _ptr(state), _ptr(conv_state), _ptr(x_new), _ptr(dt_new), _ptr(B_new), _ptr(C_new),
                                          _ptr(A), _ptr(D), int(k_draft), ctypes.byref(io)))


def mamba_spec_verify_host(ctx, state, conv_state, x, dt, B, C, A, D, n_prev_accepted, k_draft, io: IO) -> None:
    _check(ctx, lib.mamba_spec_verify_host(ctx, _ptr(state), _ptr(conv_state), _ptr(x), _ptr(dt), _ptr(B), _ptr(C),
                                           _ptr(A), _ptr(D), _ptr(n_prev_accepted), int(k_draft), ctypes.byref(io)))


def mamba_spec_verify_host_static(cfg: Config, state, conv_state, x, dt, B, C, A, D, n_prev_accepted, k_draft, io: IO,
                                  device_flags=None) -> None:
    """Context-free, allocation-free variant of ``mamba_spec_verify_host`` (host slabs staged through the
    library's built-in 8 MiB device array); ``device_flags`` is a host int32 tensor or None."""
    rc = lib.mamba_spec_verify_host_static(ctypes.byref(cfg), _ptr(state), _ptr(conv_state), _ptr(x), _ptr(dt), _ptr(B),
                                           _ptr(C), _ptr(A), _ptr(D), _ptr(n_prev_accepted), int(k_draft), ctypes.byref(io),
                                           _ptr(device_flags))
    if rc != OK:
        raise MambaSpecError(rc, lib.mamba_spec_last_error(None).decode())


def mamba_spec_commit(ctx, accept_len, batch, stream=None) -> None:
    _check(ctx, lib.mamba_spec_commit(ctx, _ptr(accept_len), int(batch), stream))


def mamba_spec_status(ctx) -> int:
    out = _i32()
    _check(ctx, lib.mamba_spec_status(ctx, ctypes.byref(out)))
    return out.value


def mamba_spec_get_n_prev(ctx, batch):
    buf = (_i32 * batch)()
    _check(ctx, lib.mamba_spec_get_n_prev(ctx, buf, batch))
    return list(buf)


def mamba_spec_get_selection(ctx, batch):
    buf = (_i32 * batch)()
    _check(ctx, lib.mamba_spec_get_selection(ctx, buf, batch))
    return list(buf)


def mamba_spec_describe_plan(cfg: Config, batch, t_max, k_draft, sm_count=0, smem_per_block=0) -> str:
    """Which kernel and launch plan a call of this shape gets (host logic only)."""
    buf = ctypes.create_string_buffer(256)
    rc = lib.mamba_spec_describe_plan(ctypes.byref(cfg), batch, t_max, k_draft, sm_count, smem_per_block, buf, 256)
    if rc != OK:
        raise MambaSpecError(rc, lib.mamba_spec_last_error(None).decode())
    return buf.value.decode()


def mamba_spec_launch_count(ctx) -> int:
    return lib.mamba_spec_launch_count(ctx)


def mamba_spec_last_kernel(ctx) -> str:
    return lib.mamba_spec_last_kernel(ctx).decode()


def mamba_spec_last_error(ctx=None) -> str:
    return lib.mamba_spec_last_error(ctx).decode()


def mamba_spec_destroy(ctx) -> None:
    lib.mamba_spec_destroy(ctx)


class Verifier:
    """Keeps one context; ``verify`` takes torch CUDA tensors and launches on the current stream."""

    def __init__(self, batch_max, H, P, N, GB, GC, W, k_max, act="bf16", flags=FLAG_GATE | FLAG_CONV_SILU,
                 n_layers=1, device=0, kernel=KERNEL_AUTO):
        self.cfg = Config(batch_max, n_layers, H, P, N, GB, GC, W, k_max,
                          DTYPE_BF16 if act == "bf16" else DTYPE_F32, flags, device, kernel)
        self.act_dtype = torch.bfloat16 if act == "bf16" else torch.float32
        self.ctx = mamba_spec_init(self.cfg)

    def close(self):
        if self.ctx:
            mamba_spec_destroy(self.ctx)
            self.ctx = None

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass

    def _io(self, conv_w, conv_b, z, y, batch, layer, t_max, stream, state_k=None, conv_state_k=None, dt_bias=None,
            norm_weight=None, norm_eps=0.0, conv_bc=None):
        if stream is None:
            stream = torch.cuda.current_stream().cuda_stream
        if norm_weight is not None:
            chan = self.cfg.n_heads * self.cfg.head_dim
            if not norm_weight.is_cuda or norm_weight.dtype != torch.float32 or tuple(norm_weight.shape) != (chan,) or \
                    not norm_weight.is_contiguous():
                raise ValueError(f"norm_weight: want contiguous CUDA torch.float32 ({chan},)")
        return IO(_ptr(conv_w), _ptr(conv_b), _ptr(z), _ptr(y), batch, layer, t_max, stream, _ptr(state_k),
                  _ptr(conv_state_k), _ptr(dt_bias), _ptr(norm_weight), float(norm_eps), *self._conv_bc(conv_bc, batch))

    def _conv_bc(self, conv_bc, batch):
        """(window, taps, bias) of the conv over the B and C channels as three pointers, shapes checked."""
        if conv_bc is None:
            return None, None, None
        c = self.cfg
        ch = (c.n_groups_b + c.n_groups_c) * c.d_state
        window, taps, bias = conv_bc
        for name, t, dtype, shape in (("conv_state_bc", window, self.act_dtype, (batch, c.conv_width - 1, ch)),
                                      ("conv_w_bc", taps, torch.float32, (ch, c.conv_width)), ("conv_b_bc", bias, torch.float32, (ch,))):
            if not t.is_cuda or t.dtype != dtype or tuple(t.shape) != shape or not t.is_contiguous():
                raise ValueError(f"{name}: want contiguous CUDA {dtype} {shape}, got {t.dtype} {tuple(t.shape)}")
        return _ptr(window), _ptr(taps), _ptr(bias)

    def verify(self, state, conv_state, x, dt, B, C, A, D, conv_w, conv_b, z, y, n_prev, k, layer=0, stream=None,
               state_k=None, conv_state_k=None, dt_bias=None, norm_weight=None, norm_eps=0.0, conv_bc=None):
        c = self.cfg
        batch, t_max = x.shape[0], x.shape[1]
        m1 = bool(c.flags & FLAG_MAMBA1)
        chan = c.n_heads * c.head_dim
        want = {
            "state": (state, torch.float32, (batch, c.n_heads, c.head_dim, c.d_state)),
            "conv_state": (conv_state, self.act_dtype, (batch, c.conv_width - 1, c.n_heads * c.head_dim)),
            "x": (x, self.act_dtype, (batch, t_max, c.n_heads, c.head_dim)),
            "dt": (dt, self.act_dtype, (batch, t_max, chan if m1 else c.n_heads)),
            "B": (B, self.act_dtype, (batch, t_max, c.n_groups_b, c.d_state)),
            "C": (C, self.act_dtype, (batch, t_max, c.n_groups_c, c.d_state)),
            "A": (A, torch.float32, (chan, c.d_state) if m1 else (c.n_heads,)),
            "D": (D, torch.float32, (chan,) if m1 else (c.n_heads,)),
            "conv_w": (conv_w, torch.float32, (c.n_heads * c.head_dim, c.conv_width)),
            "conv_b": (conv_b, torch.float32, (c.n_heads * c.head_dim,)),
            "y": (y, torch.float32 if c.flags & FLAG_Y_F32 else self.act_dtype, (batch, t_max, c.n_heads, c.head_dim)),
        }
        if z is not None:
            want["z"] = (z, self.act_dtype, (batch, t_max, c.n_heads, c.head_dim))
        if n_prev is not None:
            want["n_prev"] = (n_prev, torch.int32, (batch,))
        if c.flags & FLAG_STATE_K:   # second snapshot: the cache after all tokens of the call
            want["state_k"] = (state_k, torch.float32, (batch, c.n_heads, c.head_dim, c.d_state))
            want["conv_state_k"] = (conv_state_k, self.act_dtype, (batch, c.conv_width - 1, c.n_heads * c.head_dim))
        for name, (t, dtype, shape) in want.items():
            if not t.is_cuda or t.dtype != dtype or tuple(t.shape) != shape or not t.is_contiguous():
                raise ValueError(f"{name}: want contiguous CUDA {dtype} {shape}, got {t.dtype} {tuple(t.shape)} "
                                 f"cuda={t.is_cuda} contiguous={t.is_contiguous()}")
        if dt_bias is not None:
            want["dt_bias"] = (dt_bias, torch.float32, (chan,) if m1 else (c.n_heads,))
        for name in ("dt_bias",):
            if name in want:
                t, dtype, shape = want[name]
                if not t.is_cuda or t.dtype != dtype or tuple(t.shape) != shape or not t.is_contiguous():
                    raise ValueError(f"{name}: want contiguous CUDA {dtype} {shape}")
        io = self._io(conv_w, conv_b, z, y, batch, layer, t_max, stream, state_k, conv_state_k, dt_bias, norm_weight, norm_eps, conv_bc)
        mamba_spec_verify(self.ctx, state, conv_state, x, dt, B, C, A, D, n_prev, k, io)

    def verify_new(self, state, conv_state, x_new, dt_new, B_new, C_new, A, D, conv_w, conv_b, z_new, y_new, k, layer=0,
                   stream=None, state_k=None, conv_state_k=None, dt_bias=None, norm_weight=None, norm_eps=0.0):
        """Only the k new rows of every sequence ([batch, k, ...]); replayed rows come from the library's row store."""
        batch = y_new.shape[0]
        io = self._io(conv_w, conv_b, z_new, y_new, batch, layer, 0, stream, state_k, conv_state_k, dt_bias, norm_weight, norm_eps)
        mamba_spec_verify_new(self.ctx, state, conv_state, x_new, dt_new, B_new, C_new, A, D, k, io)

    def commit(self, accept_len, stream=None):
        if stream is None:
            stream = torch.cuda.current_stream().cuda_stream
        mamba_spec_commit(self.ctx, accept_len, accept_len.shape[0], stream)

    def status(self) -> int:
        return mamba_spec_status(self.ctx)

    def selection(self, batch):
        return mamba_spec_get_selection(self.ctx, batch)

    @property
    def last_kernel(self) -> str:
        return mamba_spec_last_kernel(self.ctx)

    @property
    def launches(self) -> int:
        return mamba_spec_launch_count(self.ctx)
