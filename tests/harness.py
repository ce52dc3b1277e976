"""Test plumbing shared by the GPU parity tests: moves seeded inputs to the device, runs the
C-ABI path and the fp64 oracle on the same buffers, and measures relative L2 error.

Nothing here computes any part of the method; the oracle never sees a value produced by
the CUDA path (both are always started from the same seeded cache and token rows).
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2408_15237_b200 import synth

TOL = {"bf16": 2e-3, "fp32": 1e-5}   # max relative L2 error on y and on the committed state


def act_dtype(s):
    return torch.bfloat16 if s.act == "bf16" else torch.float32


def dev(a, dtype):
    """numpy float32 array (values exactly representable in ``dtype``) -> CUDA tensor."""
    return torch.from_numpy(np.ascontiguousarray(a)).to(device="cuda", dtype=dtype)


def rel_l2(got, want):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    den = np.linalg.norm(want)
    num = np.linalg.norm(got - want)
    return num / den if den > 0 else num


def make_verifier(s, kernel=0, batch_max=None, k_max=None, n_layers=None, y_f32=False):
    from paper_2408_15237_b200 import binding
    flags = s.flags | (synth.FLAG_Y_F32 if y_f32 else 0)
    return binding.Verifier(batch_max or s.Bt, s.H, s.P, s.N, s.GB, s.GC, s.W, k_max if k_max is not None else s.k,
                            act=s.act, flags=flags, n_layers=n_layers or s.n_layers, kernel=kernel)


class Layer:
    """One layer's parameters and cache on both sides (numpy fp64 for the oracle, CUDA tensors for the library)."""

    def __init__(self, s, layer=0):
        self.s = s
        A, D, cw, cb = synth.layer_params(s, layer)
        st, cv = synth.initial_cache(s, layer)
        self.np = dict(A=A, D=D, cw=cw, cb=cb)
        self.o_state, self.o_conv = st.astype(np.float64), cv.astype(np.float64)
        self.A, self.D = dev(A, torch.float32), dev(D, torch.float32)
        self.cw, self.cb = dev(cw, torch.float32), dev(cb, torch.float32)
        self.state, self.conv = dev(st, torch.float32), dev(cv, act_dtype(s))
        self.bc = None
        if s.flags & synth.FLAG_CONV_BC:
            taps, bias, window = synth.conv_bc_params(s, layer)
            self.bc = dict(taps=taps, bias=bias, o_window=window.astype(np.float64),
                           dev=(dev(window, act_dtype(s)), dev(taps, torch.float32), dev(bias, torch.float32)))
        self.norm = None
        if s.flags & synth.FLAG_GATED_RMSNORM:
            w, eps = synth.norm_params(s, layer)
            self.norm = (w, eps, dev(w, torch.float32))

    def gpu_verify(self, ver, batch, k, y=None, n_prev="given", layer=0):
        s = self.s
        ad = act_dtype(s)
        t = {n: dev(batch[n], ad) for n in ("x", "z", "dt", "B", "C")}
        if y is None:
            y = torch.full(t["x"].shape, float("nan"), device="cuda",
                           dtype=torch.float32 if ver.cfg.flags & synth.FLAG_Y_F32 else ad)
        npv = dev(batch["n_prev"], torch.int32) if n_prev == "given" else None
        z = t["z"] if s.flags & synth.FLAG_GATE else None
        kw = dict(norm_weight=self.norm[2], norm_eps=self.norm[1]) if self.norm else {}
        if self.bc:
            kw["conv_bc"] = self.bc["dev"]
        ver.verify(self.state, self.conv, t["x"], t["dt"], t["B"], t["C"], self.A, self.D, self.cw, self.cb, z, y,
                   npv, k, layer=layer, **kw)
        torch.cuda.synchronize()
        return y

    def oracle_verify(self, batch, k, threads=None):
        s, p = self.s, self.np
        z = batch["z"] if s.flags & synth.FLAG_GATE else None
        core = s.flags & (synth.FLAG_GATE | synth.FLAG_CONV_SILU)
        if self.bc:
            y, self.o_state, self.o_conv, self.bc["o_window"] = oracle.verify_conv_bc(
                self.o_state, self.o_conv, self.bc["o_window"], batch["x"], batch["dt"], batch["B"], batch["C"], p["A"], p["D"],
                p["cw"], p["cb"], self.bc["taps"], self.bc["bias"], z, batch["n_prev"], k, core, threads=threads or oracle.host_threads())
        else:
            y, self.o_state, self.o_conv = oracle.verify(
                self.o_state, self.o_conv, batch["x"], batch["dt"], batch["B"], batch["C"], p["A"], p["D"], p["cw"],
                p["cb"], z, batch["n_prev"], k, core, threads=threads or oracle.host_threads())
        if self.norm:
            y = oracle.gated_rmsnorm(y, self.norm[0], self.norm[1])
        return y

    def check(self, y_gpu, y_ref, tol, what=""):
        """Relative L2 of y (valid rows only; the rest must still be NaN) and of the cache."""
        yg = y_gpu.float().cpu().numpy().astype(np.float64)
        valid = ~np.isnan(y_ref)
        assert np.isnan(yg[~valid]).all(), f"{what}: rows beyond T_b were written"
        assert not np.isnan(yg[valid]).any(), f"{what}: NaN in a valid output row"
        e_y = rel_l2(yg[valid], y_ref[valid])
        e_s = rel_l2(self.state.cpu().numpy(), self.o_state)
        e_c = np.abs(self.conv.float().cpu().numpy().astype(np.float64) - self.o_conv).max() if self.o_conv.size else 0.0
        if self.bc:   # the window of the conv over B and C is a copy of input rows: exact
            e_c = max(e_c, np.abs(self.bc["dev"][0].float().cpu().numpy().astype(np.float64) - self.bc["o_window"]).max())
        if y_gpu.dtype == torch.bfloat16:
            # y is a bf16 code: both sides take the rounding in the same precision.  Rounding the exact
            # output to bf16 costs 1.4e-3 .. 2.4e-3 relative L2 by itself on these workloads, so the
            # tolerance is applied against the oracle rounded to bf16, and the distance to the unrounded
            # oracle may exceed that rounding floor by no more than a tenth of the tolerance.
            y_ref_q = synth.round_bf16(np.nan_to_num(y_ref).astype(np.float32)).astype(np.float64)
            floor = rel_l2(y_ref_q[valid], y_ref[valid])
            e_q = rel_l2(yg[valid], y_ref_q[valid])
            assert e_q <= tol, f"{what}: y rel L2 against the bf16-rounded oracle {e_q:.3e} > {tol}"
            assert e_y <= floor + 0.1 * tol, f"{what}: y rel L2 {e_y:.3e} vs rounding floor {floor:.3e}"
            # and the stated tolerance taken literally, against the unrounded oracle, wherever rounding the exact output
            # to bf16 leaves room for it.  That rounding alone costs 1.4e-3 .. 1.8e-3 on the large workloads and
            # 2.0e-3 .. 2.4e-3 where few values are compared (batch 1 with two drafts, the small edge shapes): there
            # a perfect kernel exceeds 2e-3, and the two checks above and the fp32-output tests stand in.
            self.last_floor = floor
            if floor <= 0.9 * tol:
                assert e_y <= tol, f"{what}: y rel L2 against the unrounded oracle {e_y:.3e} > {tol}"
            self.last_unrounded = e_y
            e_y = e_q
        else:
            assert e_y <= tol, f"{what}: y rel L2 {e_y:.3e} > {tol}"
        assert e_s <= tol, f"{what}: state rel L2 {e_s:.3e} > {tol}"
        assert e_c == 0.0, f"{what}: conv window differs by {e_c}"
        # per sequence as well: one bad sequence must not hide in the batch norm
        for b in range(yg.shape[0]):
            e = rel_l2(self.state[b].cpu().numpy(), self.o_state[b])
            assert e <= tol, f"{what}: state rel L2 of sequence {b} is {e:.3e}"
            if not valid[b].any():
                continue
            got, want = yg[b][valid[b]], y_ref[b][valid[b]]
            if y_gpu.dtype == torch.bfloat16:
                # A bf16 store alone costs up to 2^-8 relative per element (1.4e-3 .. 2.4e-3 relative L2 on these
                # outputs), so a small tensor can sit above 2e-3 through rounding only.  Per sequence the check
                # is therefore elementwise: every output is the correctly rounded oracle value up to fp32 noise.
                bound = 2.0 ** -8 * np.abs(want) + 2e-5 * np.sqrt(np.mean(want ** 2))
                bad = np.abs(got - want) > bound
                assert not bad.any(), f"{what}: sequence {b}: {bad.sum()} outputs are not the rounded oracle value"
            else:
                e = rel_l2(got, want)
                assert e <= tol, f"{what}: y rel L2 of sequence {b} is {e:.3e}"
        return e_y, e_s


def run_rounds(s, rounds, kernel=0, layer=0, first_j=None, accept=None, final_flush=False, y_f32=False, tol=None):
    """Runs ``rounds`` speculation rounds of one layer on both sides, checking after every round."""
    tol = tol or TOL[s.act]
    ver = make_verifier(s, kernel, y_f32=y_f32)
    lay = Layer(s, layer)
    fj = s.first_j if first_j is None else first_j
    stream = synth.token_stream(s, layer, rounds * s.k + s.k + fj + 1)
    r = synth.Rounds(s, stream, first_j=fj)
    worst = (0.0, 0.0)
    run_rounds.worst_unrounded = 0.0   # largest rel L2 of a bf16 y against the UNROUNDED oracle (the figure the tolerance names)
    for rd in range(rounds):
        b = r.batch()
        y_gpu = lay.gpu_verify(ver, b, s.k)
        y_ref = lay.oracle_verify(b, s.k)
        e = lay.check(y_gpu, y_ref, tol, f"{s.name} round {rd} [{ver.last_kernel}]")
        worst = (max(worst[0], e[0]), max(worst[1], e[1]))
        run_rounds.worst_unrounded = max(run_rounds.worst_unrounded, getattr(lay, "last_unrounded", e[0]))
        a = synth.acceptance(s, rd) if accept is None else np.asarray(accept(rd), dtype=np.int32)
        r.accept(a)
    if final_flush:
        b = r.batch()
        y_gpu = lay.gpu_verify(ver, b, 0)
        y_ref = lay.oracle_verify(b, 0)
        lay.check(y_gpu, y_ref, tol, f"{s.name} flush [{ver.last_kernel}]")
    assert ver.status() == 0
    name = ver.last_kernel
    ver.close()
    return worst, name
