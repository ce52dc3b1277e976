"""TEST INFRASTRUCTURE ONLY: Python face of the fp64 CPU oracle (``oracle.c``).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It never imports the CUDA package and shares no code with it.

The C file is compiled with gcc on first use (no fast-math, no FMA contraction)
into ``oracle/_build/``; arrays cross as contiguous float64 / int32 numpy
buffers.  All functions follow the paper's statement of the recurrence (Eq. 1),
its on-the-fly discretisation (Sec. 2.2) and the multi-step verification call
(Sec. 4.2, Sec. 4.3); see the header of ``oracle.c`` for the readings taken.
"""
from __future__ import annotations

import ctypes
import hashlib
import os
import subprocess
from pathlib import Path

import numpy as np

FLAG_GATE = 1
FLAG_CONV_SILU = 2

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "oracle.c"
_LIB = None


class _Dims(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("Bt", "Tmax", "H", "P", "N", "GB", "GC", "W", "flags")]


def build(force: bool = False) -> Path:
    """Compile ``oracle.c`` into a shared library named after its content hash."""
    digest = hashlib.sha256(_SRC.read_bytes()).hexdigest()[:12]
    out_dir = _HERE / "_build"
    out = out_dir / f"liboracle_{digest}.so"
    if out.exists() and not force:
        return out
    out_dir.mkdir(exist_ok=True)
    tmp = out_dir / f".tmp_{os.getpid()}_{digest}.so"
    cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
           "-shared", "-fPIC", str(_SRC), "-o", str(tmp), "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, out)
    return out


def _lib():
    global _LIB
    if _LIB is None:
        lib = ctypes.CDLL(str(build()))
        dp, ip = ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_int32)
        lib.oracle_verify.restype = ctypes.c_int
        lib.oracle_verify.argtypes = [ctypes.POINTER(_Dims), ctypes.c_int32, ip] + [dp] * 14 + [ctypes.c_int32]
        lib.oracle_step.restype = ctypes.c_int
        lib.oracle_step.argtypes = [ctypes.POINTER(_Dims)] + [dp] * 12 + [ip]
        lib.oracle_sequential.restype = ctypes.c_int
        lib.oracle_sequential.argtypes = [ctypes.POINTER(_Dims), ctypes.c_int32, ip] + [dp] * 12 + [ctypes.c_int32]
        lib.oracle_verify_m1.restype = ctypes.c_int
        lib.oracle_verify_m1.argtypes = [ctypes.POINTER(_Dims), ctypes.c_int32, ip] + [dp] * 14 + [ctypes.c_int32]
        lib.oracle_step_m1.restype = ctypes.c_int
        lib.oracle_step_m1.argtypes = [ctypes.POINTER(_Dims)] + [dp] * 12
        _LIB = lib
    return _LIB


def _f64(a, shape=None):
    a = np.ascontiguousarray(np.asarray(a, dtype=np.float64))
    if shape is not None and tuple(a.shape) != tuple(shape):
        raise ValueError(f"expected shape {tuple(shape)}, got {a.shape}")
    return a


def _dp(a):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _ip(a):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))


def host_threads() -> int:
    """Number of host cores this process may run on."""
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:  # pragma: no cover
        return os.cpu_count() or 1


def _dims(state, conv_state, Bm, Cm, Tmax, flags):
    Bt, H, P, N = state.shape
    W = conv_state.shape[1] + 1
    if conv_state.shape != (Bt, W - 1, H * P):
        raise ValueError(f"conv_state shape {conv_state.shape}")
    return _Dims(Bt, Tmax, H, P, N, Bm.shape[-2], Cm.shape[-2], W, flags)


def verify(state, conv_state, x, dt, Bm, Cm, A, D, conv_w, conv_b, z, n_prev, k, flags, threads=1):
    """Multi-step verification (Sec. 4.2 MultiStep; Sec. 4.3 replay + draft + caching).

    Returns ``(y, state_out, conv_state_out)``; ``y`` rows at and beyond
    ``n_prev[b] + k`` are NaN (never written).
    """
    state, conv_state = _f64(state), _f64(conv_state)
    Bt, H, P, N = state.shape
    x = _f64(x)
    Tmax = x.shape[1]
    Bm, Cm = _f64(Bm), _f64(Cm)
    d = _dims(state, conv_state, Bm, Cm, Tmax, flags)
    x = _f64(x, (Bt, Tmax, H, P))
    dt = _f64(dt, (Bt, Tmax, H))
    Bm = _f64(Bm, (Bt, Tmax, d.GB, N))
    Cm = _f64(Cm, (Bt, Tmax, d.GC, N))
    A, D = _f64(A, (H,)), _f64(D, (H,))
    conv_w, conv_b = _f64(conv_w, (H * P, d.W)), _f64(conv_b, (H * P,))
    z = None if z is None else _f64(z, (Bt, Tmax, H, P))
    n_prev = np.ascontiguousarray(np.asarray(n_prev, dtype=np.int32))
    if n_prev.shape != (Bt,):
        raise ValueError("n_prev shape")
    y = np.full((Bt, Tmax, H, P), np.nan, dtype=np.float64)
    s_out, c_out = np.empty_like(state), np.empty_like(conv_state)
    rc = _lib().oracle_verify(ctypes.byref(d), int(k), _ip(n_prev), _dp(state), _dp(conv_state), _dp(x), _dp(dt),
                              _dp(Bm), _dp(Cm), _dp(A), _dp(D), _dp(conv_w), _dp(conv_b), _dp(z),
                              _dp(y), _dp(s_out), _dp(c_out), int(threads))
    if rc != 0:
        raise ValueError("oracle_verify: n_prev out of range for Tmax")
    return y, s_out, c_out


def step(state, conv_state, x1, dt1, B1, C1, A, D, conv_w, conv_b, z1, flags, active=None):
    """One decoding step for every (active) sequence (Eq. 1); returns ``(y1, state, conv_state)`` as new arrays."""
    state, conv_state = _f64(state).copy(), _f64(conv_state).copy()
    Bt, H, P, N = state.shape
    B1, C1 = _f64(B1), _f64(C1)
    d = _dims(state, conv_state, B1, C1, 1, flags)
    x1, dt1 = _f64(x1, (Bt, H, P)), _f64(dt1, (Bt, H))
    B1, C1 = _f64(B1, (Bt, d.GB, N)), _f64(C1, (Bt, d.GC, N))
    A, D = _f64(A, (H,)), _f64(D, (H,))
    conv_w, conv_b = _f64(conv_w, (H * P, d.W)), _f64(conv_b, (H * P,))
    z1 = None if z1 is None else _f64(z1, (Bt, H, P))
    act = None if active is None else np.ascontiguousarray(np.asarray(active, dtype=np.int32))
    y1 = np.full((Bt, H, P), np.nan, dtype=np.float64)
    _lib().oracle_step(ctypes.byref(d), _dp(state), _dp(conv_state), _dp(x1), _dp(dt1), _dp(B1), _dp(C1),
                       _dp(A), _dp(D), _dp(conv_w), _dp(conv_b), _dp(z1), _dp(y1), _ip(act))
    return y1, state, conv_state


def sequential(state, conv_state, x, dt, Bm, Cm, A, D, conv_w, conv_b, z, lengths, flags, threads=1):
    """Plain run over a token stream with no speculation (Alg. 2's ground truth).

    ``x`` is ``[Bt, L, H, P]``; sequence ``b`` consumes ``lengths[b]`` tokens.
    Returns ``(y, state, conv_state)``; unused ``y`` rows are NaN.
    """
    state, conv_state = _f64(state).copy(), _f64(conv_state).copy()
    Bt, H, P, N = state.shape
    x = _f64(x)
    L = x.shape[1]
    Bm, Cm = _f64(Bm), _f64(Cm)
    d = _dims(state, conv_state, Bm, Cm, L, flags)
    x, dt = _f64(x, (Bt, L, H, P)), _f64(dt, (Bt, L, H))
    Bm, Cm = _f64(Bm, (Bt, L, d.GB, N)), _f64(Cm, (Bt, L, d.GC, N))
    A, D = _f64(A, (H,)), _f64(D, (H,))
    conv_w, conv_b = _f64(conv_w, (H * P, d.W)), _f64(conv_b, (H * P,))
    z = None if z is None else _f64(z, (Bt, L, H, P))
    lengths = np.ascontiguousarray(np.asarray(lengths, dtype=np.int32))
    y = np.full((Bt, L, H, P), np.nan, dtype=np.float64)
    rc = _lib().oracle_sequential(ctypes.byref(d), int(L), _ip(lengths), _dp(state), _dp(conv_state), _dp(x), _dp(dt),
                                  _dp(Bm), _dp(Cm), _dp(A), _dp(D), _dp(conv_w), _dp(conv_b), _dp(z), _dp(y),
                                  int(threads))
    if rc != 0:
        raise ValueError("oracle_sequential: lengths out of range")
    return y, state, conv_state


def softplus_dt(dt_raw, bias):
    """The sampling interval from its raw value: ``softplus(dt_raw + bias)`` with the bias broadcast over the
    last axis (Sec. 2.2: the intervals come out of a network; a softplus keeps them positive)."""
    v = np.asarray(dt_raw, dtype=np.float64) + np.asarray(bias, dtype=np.float64)
    return np.where(v > 30.0, v, np.log1p(np.exp(np.minimum(v, 30.0))))


def conv_rows(rows, window, taps, bias, n_prev, k, silu):
    """The rolling depthwise causal conv of the Mamba block (Sec. 4.3, footnote) over the token rows of any channel
    set: ``rows [Bt, Tmax, Ch]`` are the inputs of this call, ``window [Bt, W-1, Ch]`` the last W-1 inputs before
    them (oldest first), ``taps [Ch, W]`` (tap W-1 multiplies the current token), ``bias [Ch]``.  Returns the
    outputs ``[Bt, Tmax, Ch]`` (NaN at and beyond ``n_prev[b] + k``) and the window after the first ``n_prev[b]``
    tokens, i.e. at the newly verified position (unchanged where ``n_prev[b] = 0``)."""
    rows, window = np.asarray(rows, dtype=np.float64), np.asarray(window, dtype=np.float64)
    taps, bias = np.asarray(taps, dtype=np.float64), np.asarray(bias, dtype=np.float64)
    Bt, Tmax, Ch = rows.shape
    W = taps.shape[1]
    if window.shape != (Bt, W - 1, Ch) or taps.shape != (Ch, W) or bias.shape != (Ch,):
        raise ValueError("conv_rows: shapes")
    out = np.full((Bt, Tmax, Ch), np.nan)
    win_out = window.copy()
    for b in range(Bt):
        j, T = int(n_prev[b]), int(n_prev[b]) + int(k)
        hist = [window[b, w] for w in range(W - 1)]          # the W-1 inputs before token 0
        for t in range(T):
            hist.append(rows[b, t])
            acc = bias.copy()
            for w in range(W):
                acc = acc + taps[:, w] * hist[t + w]          # hist[t + w] is input t - (W-1) + w
            out[b, t] = acc / (1.0 + np.exp(-acc)) if silu else acc
            if t == j - 1:
                for w in range(W - 1):
                    win_out[b, w] = hist[t + 1 + w]           # the last W-1 inputs up to token j-1
    return out, win_out


def verify_conv_bc(state, conv_state, conv_state_bc, x, dt, Bm, Cm, A, D, conv_w, conv_b, conv_w_bc, conv_b_bc, z, n_prev, k,
                   flags, threads=1):
    """The verification call for blocks whose conv runs over x, B and C together (the Mamba-2 block of the hybrid
    Mamba2 models, Sec. 5): the B and C rows pass through their own depthwise causal conv (channels: the G_B*N
    columns of B, then the G_C*N columns of C; own taps, bias and rolling window) and the same activation as x
    before they enter the recurrence.  Returns ``(y, state_out, conv_state_out, conv_state_bc_out)``.
    Not in the paper's text (parity unpinned by the paper); the conv itself is the one of Sec. 4.3."""
    Bm, Cm = np.asarray(Bm, dtype=np.float64), np.asarray(Cm, dtype=np.float64)
    Bt, Tmax, GB, N = Bm.shape
    GC = Cm.shape[2]
    rows = np.concatenate([Bm.reshape(Bt, Tmax, GB * N), Cm.reshape(Bt, Tmax, GC * N)], axis=2)
    out, win = conv_rows(rows, conv_state_bc, conv_w_bc, conv_b_bc, n_prev, k, bool(flags & 2))
    out = np.nan_to_num(out)     # rows beyond T_b are never read by the recurrence
    Bc = out[:, :, :GB * N].reshape(Bt, Tmax, GB, N)
    Cc = out[:, :, GB * N:].reshape(Bt, Tmax, GC, N)
    y, s_out, c_out = verify(state, conv_state, x, dt, Bc, Cc, A, D, conv_w, conv_b, z, n_prev, k, flags, threads=threads)
    return y, s_out, c_out, win


def gated_rmsnorm(y, weight, eps):
    """The output normalisation of the Mamba-2 blocks that the hybrid Mamba2 models (Sec. 5) are made of: with
    ``y`` the gated output of the verification call, ``[..., H, P]``, every token row is scaled to unit mean
    square over its ``H*P`` channels and multiplied by a learned per-channel weight,
    ``out[c] = weight[c] * y[c] / sqrt(mean_c(y[c]^2) + eps)``.  Rows that hold NaN (padding) stay NaN.
    The paper does not print this formula; it is the published Mamba-2 block's (parity unpinned by the paper)."""
    y = np.asarray(y, dtype=np.float64)
    w = np.asarray(weight, dtype=np.float64).reshape(-1)
    rows = y.reshape(-1, y.shape[-2] * y.shape[-1])
    if rows.shape[1] != w.shape[0]:
        raise ValueError("gated_rmsnorm: weight must have H*P entries")
    out = np.empty_like(rows)
    for r in range(rows.shape[0]):          # one token at a time, as the definition reads
        mean_square = np.sum(rows[r] * rows[r]) / rows.shape[1]
        out[r] = w * rows[r] / np.sqrt(mean_square + float(eps))
    return out.reshape(y.shape)


def verify_m1(state, conv_state, x, dt, Bm, Cm, A, D, conv_w, conv_b, z, n_prev, k, flags, threads=1):
    """Multi-step verification in the Mamba-1 parameterisation (Algorithm 1; Sec. 2.2): ``dt`` is
    ``[Bt, Tmax, H*P]``, ``A`` is ``[H*P, N]``, ``D`` is ``[H*P]``.  Returns ``(y, state_out, conv_state_out)``."""
    state, conv_state = _f64(state), _f64(conv_state)
    Bt, H, P, N = state.shape
    if N > 1024 or conv_state.shape[1] > 16:
        raise ValueError("oracle_verify_m1 keeps a row of at most 1024 columns and 16 window slots on the stack")
    x = _f64(x)
    Tmax = x.shape[1]
    Bm, Cm = _f64(Bm), _f64(Cm)
    d = _dims(state, conv_state, Bm, Cm, Tmax, flags)
    x = _f64(x, (Bt, Tmax, H, P))
    dt = _f64(dt, (Bt, Tmax, H * P))
    Bm, Cm = _f64(Bm, (Bt, Tmax, d.GB, N)), _f64(Cm, (Bt, Tmax, d.GC, N))
    A, D = _f64(A, (H * P, N)), _f64(D, (H * P,))
    conv_w, conv_b = _f64(conv_w, (H * P, d.W)), _f64(conv_b, (H * P,))
    z = None if z is None else _f64(z, (Bt, Tmax, H, P))
    n_prev = np.ascontiguousarray(np.asarray(n_prev, dtype=np.int32))
    if n_prev.shape != (Bt,):
        raise ValueError("n_prev shape")
    y = np.full((Bt, Tmax, H, P), np.nan, dtype=np.float64)
    s_out, c_out = np.empty_like(state), np.empty_like(conv_state)
    rc = _lib().oracle_verify_m1(ctypes.byref(d), int(k), _ip(n_prev), _dp(state), _dp(conv_state), _dp(x), _dp(dt),
                                 _dp(Bm), _dp(Cm), _dp(A), _dp(D), _dp(conv_w), _dp(conv_b), _dp(z),
                                 _dp(y), _dp(s_out), _dp(c_out), int(threads))
    if rc != 0:
        raise ValueError("oracle_verify_m1: n_prev out of range for Tmax")
    return y, s_out, c_out


def step_m1(state, conv_state, x1, dt1, B1, C1, A, D, conv_w, conv_b, z1, flags):
    """One decoding step of every sequence in the Mamba-1 parameterisation; returns ``(y1, state, conv_state)``."""
    state, conv_state = _f64(state).copy(), _f64(conv_state).copy()
    Bt, H, P, N = state.shape
    B1, C1 = _f64(B1), _f64(C1)
    d = _dims(state, conv_state, B1, C1, 1, flags)
    x1, dt1 = _f64(x1, (Bt, H, P)), _f64(dt1, (Bt, H * P))
    B1, C1 = _f64(B1, (Bt, d.GB, N)), _f64(C1, (Bt, d.GC, N))
    A, D = _f64(A, (H * P, N)), _f64(D, (H * P,))
    conv_w, conv_b = _f64(conv_w, (H * P, d.W)), _f64(conv_b, (H * P,))
    z1 = None if z1 is None else _f64(z1, (Bt, H, P))
    y1 = np.full((Bt, H, P), np.nan, dtype=np.float64)
    _lib().oracle_step_m1(ctypes.byref(d), _dp(state), _dp(conv_state), _dp(x1), _dp(dt1), _dp(B1), _dp(C1),
                          _dp(A), _dp(D), _dp(conv_w), _dp(conv_b), _dp(z1), _dp(y1))
    return y1, state, conv_state
