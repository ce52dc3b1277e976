"""Seeded synthetic inputs for the multi-step Mamba verification step.

This module is the only thing the CPU oracle's tests and the CUDA path's tests
share.  It draws random numbers, rounds them to the activation precision and
lays rows out; it holds none of the method's arithmetic (no convolution, no
recurrence, no decay).  Random streams are numpy Philox generators keyed by a
hash of (base seed, config, layer, tensor), so a tensor depends on nothing but
its own name.

Shapes and distributions imitate one Mamba layer of a distilled
Llama3-8B-style hybrid during speculative decoding (Sec. 4 of the paper; the
paper's prompts and checkpoints are not available, only tensor shapes and
acceptance statistics are imitated):

    x, z ~ N(0,1)          dt = softplus(N(0,1) - 2)      A_h = -exp(U(0, ln 16))
    B, C ~ N(0, 1/N)       D ~ N(0,1)                     conv_w ~ N(0, 1/W), conv_b ~ N(0, 0.1^2)
    initial state, conv window ~ N(0, 0.1^2)

Activations (x, z, dt, B, C, the conv window) are rounded to the activation
dtype (bf16 round-to-nearest-even, or left in fp32) and returned as float32
arrays holding exactly representable values; parameters and the state are fp32.
"""
from __future__ import annotations

import hashlib
from dataclasses import dataclass, replace

import numpy as np

BASE_SEED = 20240815
FLAG_GATE = 1
FLAG_CONV_SILU = 2
FLAG_Y_F32 = 4      # outputs in float32 whatever the activation dtype
FLAG_STATE_K = 8    # second snapshot: the cache after all tokens of the call
FLAG_GATED_RMSNORM = 128   # the output rows are normalised (unit mean square over H*P channels) and weighted
FLAG_CONV_BC = 256         # the B and C rows pass through a depthwise conv of their own before the recurrence


@dataclass(frozen=True)
class Shape:
    """One layer's problem shape.  ``act`` is 'fp32' or 'bf16'."""
    name: str
    Bt: int
    H: int
    P: int
    N: int
    GB: int
    GC: int
    W: int
    k: int
    act: str
    flags: int = FLAG_GATE | FLAG_CONV_SILU
    n_layers: int = 1
    rounds: int = 1
    accept: str = "uniform"       # 'uniform' on {0..k}, or 'geometric'
    accept_p: float = 0.0
    first_j: int = 0
    t_rows: int = 0               # token rows per sequence in a call; 0 = 2k (k replayed + k draft at most)
    k_prev: int = 0               # most tokens that can be pending (accepted elsewhere, e.g. by a verifier); 0 = k

    @property
    def t_max(self) -> int:
        return self.t_rows if self.t_rows > 0 else 2 * self.k


def llama8b_layer(name, Bt, k, **kw) -> Shape:
    """Llama3-8B-shaped Mamba layer: 32 heads of 128 channels, state 128, B from 8 KV groups, C per head."""
    return Shape(name=name, Bt=Bt, H=32, P=128, N=128, GB=8, GC=32, W=4, k=k, act="bf16", **kw)


CONFIGS = {
    0: Shape("c0_tiny_fp32", Bt=1, H=2, P=16, N=16, GB=1, GC=2, W=4, k=4, act="fp32", rounds=20, first_j=2),
    1: llama8b_layer("c1_llama8b_b1", 1, 4),
    3: Shape("c3_small_state", Bt=32, H=64, P=64, N=64, GB=8, GC=64, W=4, k=8, act="bf16",
             accept="geometric", accept_p=0.3),
    4: llama8b_layer("c4_hybrid_stack", 16, 4, n_layers=24, rounds=200, accept="geometric", accept_p=0.4),
}
# config 2: the batch x draft-length sweep on the config-1 layer shape
SWEEP = {(bt, k): llama8b_layer(f"c2_b{bt}_k{k}", bt, k) for bt in (1, 4, 16, 64) for k in (2, 4, 8)}


def rng(*names) -> np.random.Generator:
    key = hashlib.sha256(repr((BASE_SEED,) + tuple(names)).encode()).digest()
    return np.random.Generator(np.random.Philox(key=int.from_bytes(key[:16], "little")))


def round_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result stays float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    bits = a.view(np.uint32).astype(np.uint64)
    bits = (bits + 0x7FFF + ((bits >> 16) & 1)) & 0xFFFF0000
    out = bits.astype(np.uint32).view(np.float32).reshape(a.shape)
    return np.where(np.isfinite(a), out, a).astype(np.float32)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of an array that already holds bf16-representable float32 values."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> 16).astype(np.uint16).reshape(a.shape)


def to_act(a: np.ndarray, act: str) -> np.ndarray:
    a = np.asarray(a, dtype=np.float32)
    return round_bf16(a) if act == "bf16" else a


def layer_params(s: Shape, layer: int = 0):
    """Per-layer constants: A [H] (negative), D [H], conv_w [H*P, W], conv_b [H*P]; all fp32."""
    g = rng(s.name, layer, "params")
    A = -np.exp(g.uniform(0.0, np.log(16.0), size=s.H)).astype(np.float32)
    D = g.standard_normal(s.H).astype(np.float32)
    conv_w = (g.standard_normal((s.H * s.P, s.W)) / np.sqrt(s.W)).astype(np.float32)
    conv_b = (0.1 * g.standard_normal(s.H * s.P)).astype(np.float32)
    return A, D, conv_w, conv_b


def initial_cache(s: Shape, layer: int = 0):
    """Cached SSM state [Bt,H,P,N] fp32 and conv window [Bt,W-1,H*P] in the activation precision."""
    g = rng(s.name, layer, "cache")
    state = (0.1 * g.standard_normal((s.Bt, s.H, s.P, s.N), dtype=np.float32)).astype(np.float32)
    conv = to_act(0.1 * g.standard_normal((s.Bt, s.W - 1, s.H * s.P), dtype=np.float32), s.act)
    return state, conv


def token_stream(s: Shape, layer: int, length: int):
    """A stream of ``length`` token rows per sequence: dict of x,z [Bt,L,H,P], dt [Bt,L,H], B [Bt,L,GB,N], C [Bt,L,GC,N]."""
    g = rng(s.name, layer, "stream", length)
    f32 = np.float32
    x = g.standard_normal((s.Bt, length, s.H, s.P), dtype=f32)
    z = g.standard_normal((s.Bt, length, s.H, s.P), dtype=f32)
    pre = g.standard_normal((s.Bt, length, s.H), dtype=f32) - f32(2.0)
    dt = np.log1p(np.exp(pre.astype(np.float64))).astype(f32)
    Bm = g.standard_normal((s.Bt, length, s.GB, s.N), dtype=f32) / f32(np.sqrt(s.N))
    Cm = g.standard_normal((s.Bt, length, s.GC, s.N), dtype=f32) / f32(np.sqrt(s.N))
    return {k: to_act(v, s.act) for k, v in dict(x=x, z=z, dt=dt, B=Bm, C=Cm).items()}


def acceptance(s: Shape, layer_independent_round: int) -> np.ndarray:
    """Acceptance lengths [Bt] in [0,k] for one round, independent per sequence.

    'uniform' is uniform on {0..k}; 'geometric' is min(k, G) with P(G=m)=(1-p)^m p,
    i.e. p is the per-token rejection probability; 'none' accepts nothing (every
    call then starts from the cached state: plain multi-step decoding).
    """
    g = rng(s.name, "accept", layer_independent_round)
    cap = s.k_prev if s.k_prev > 0 else s.k
    if s.accept == "none":
        return np.zeros(s.Bt, dtype=np.int32)
    if s.accept == "geometric":
        a = g.geometric(s.accept_p, size=s.Bt) - 1
        return np.minimum(a, cap).astype(np.int32)
    return g.integers(0, cap + 1, size=s.Bt).astype(np.int32)


class Rounds:
    """Bookkeeping of a speculative-decoding run over a token stream.

    ``cursor[b]`` counts the tokens of sequence b verified so far (stream rows
    [0, cursor) are accepted); ``n_prev[b]`` of them are not yet folded into the
    cached state.  ``batch()`` lays out, left-aligned, the n_prev replayed rows
    followed by the k draft rows (the next k stream rows); every other row is
    NaN so that a kernel reading padding shows up.  ``accept(a)`` moves on.
    """

    def __init__(self, s: Shape, stream: dict, first_j: int = 0, wrap: bool = False):
        self.s, self.stream, self.wrap = s, stream, wrap
        self.L = stream["x"].shape[1]
        self.cursor = np.full(s.Bt, first_j, dtype=np.int64)
        self.n_prev = np.full(s.Bt, first_j, dtype=np.int32)

    def rows(self, k=None, t_max=None) -> np.ndarray:
        """Stream row index of every slot, [Bt, t_max]; -1 marks padding.  ``k`` overrides the draft length."""
        s = self.s
        k = s.k if k is None else k
        t = np.arange(s.t_max if t_max is None else t_max)[None, :]
        start = (self.cursor - self.n_prev)[:, None]
        idx = start + t
        valid = t < (self.n_prev[:, None] + k)
        if self.wrap:
            idx = idx % self.L
        elif (idx[valid] >= self.L).any():
            raise ValueError("token stream exhausted")
        return np.where(valid, idx, -1)

    def batch(self, k=None, t_max=None) -> dict:
        idx = self.rows(k, t_max)
        out = {}
        b = np.arange(self.s.Bt)[:, None]
        for name, arr in self.stream.items():
            g = arr[b, np.maximum(idx, 0)]
            g[idx < 0] = np.nan
            out[name] = g
        out["n_prev"] = self.n_prev.copy()
        return out

    def accept(self, a: np.ndarray) -> None:
        a = np.asarray(a, dtype=np.int32)
        if (a < 0).any() or (a > self.s.k).any():
            raise ValueError("acceptance length outside [0,k]")
        self.cursor = self.cursor + a
        self.n_prev = a.copy()


def with_batch(s: Shape, Bt: int) -> Shape:
    return replace(s, Bt=Bt, name=f"{s.name}_bt{Bt}")


def conv_bc_params(s: Shape, layer: int = 0):
    """Taps [(GB+GC)*N, W], bias [(GB+GC)*N] (fp32) and the initial window [Bt, W-1, (GB+GC)*N] (activation precision)
    of the conv over the B and C channels."""
    g = rng(s.name, layer, "conv_bc")
    ch = (s.GB + s.GC) * s.N
    taps = (g.standard_normal((ch, s.W)) / np.sqrt(s.W)).astype(np.float32)
    bias = (0.1 * g.standard_normal(ch)).astype(np.float32)
    window = to_act((0.1 * g.standard_normal((s.Bt, s.W - 1, ch))).astype(np.float32), s.act)
    return taps, bias, window


def norm_params(s: Shape, layer: int = 0):
    """Weight [H*P] (fp32, around one) and eps of the output normalisation."""
    g = rng(s.name, layer, "norm")
    return (1.0 + 0.1 * g.standard_normal(s.H * s.P)).astype(np.float32), 1e-5


def m1_params(s: Shape, layer: int = 0):
    """Mamba-1 form of the per-layer constants (Algorithm 1): A [H*P, N] negative, D [H*P]; fp32."""
    g = rng(s.name, layer, "params_m1")
    A = -np.exp(g.uniform(0.0, np.log(16.0), size=(s.H * s.P, s.N))).astype(np.float32)
    D = g.standard_normal(s.H * s.P).astype(np.float32)
    return A, D


def m1_dt_stream(s: Shape, layer: int, length: int) -> np.ndarray:
    """Mamba-1 form of the sampling intervals: one per (token, channel), [Bt, L, H*P], same distribution as dt."""
    g = rng(s.name, layer, "stream_m1_dt", length)
    pre = g.standard_normal((s.Bt, length, s.H * s.P), dtype=np.float32) - np.float32(2.0)
    return to_act(np.log1p(np.exp(pre.astype(np.float64))).astype(np.float32), s.act)


def raw_dt_stream(s: Shape, layer: int, length: int, per_channel: bool = False):
    """Raw intervals (before the softplus) and their bias: dt_raw ~ N(0,1) in the activation precision, [Bt, L, H]
    ([Bt, L, H*P] per channel), bias ~ N(-2, 0.25) fp32, so that softplus(dt_raw + bias) is distributed like dt."""
    g = rng(s.name, layer, "stream_raw_dt", length, per_channel)
    n = s.H * s.P if per_channel else s.H
    raw = to_act(g.standard_normal((s.Bt, length, n), dtype=np.float32), s.act)
    bias = (np.float32(-2.0) + np.float32(0.5) * g.standard_normal(n)).astype(np.float32)
    return raw, bias
