"""GPU edge cases of the verification call: degenerate lengths, clamping, commit bookkeeping,
untouched memory, determinism, the host-buffer entry point and argument errors."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2408_15237_b200 import synth

pytestmark = pytest.mark.gpu

GENERIC, STREAM = 1, 2
SMALL = synth.Shape("edge_small", Bt=5, H=8, P=64, N=128, GB=2, GC=8, W=4, k=4, act="bf16")
SMALL64 = synth.Shape("edge_small64", Bt=3, H=8, P=32, N=64, GB=8, GC=1, W=4, k=3, act="bf16")
ODD = synth.Shape("edge_odd_fp32", Bt=2, H=3, P=12, N=40, GB=1, GC=3, W=3, k=2, act="fp32")
NOGATE = synth.Shape("edge_nogate", Bt=2, H=8, P=32, N=128, GB=1, GC=8, W=4, k=4, act="bf16", flags=0)


def H():
    import harness
    return harness


@pytest.mark.parametrize("kernel", [GENERIC, STREAM])
@pytest.mark.parametrize("case", ["none_accepted", "all_accepted", "mixed"])
def test_acceptance_patterns(kernel, case):
    h = H()
    s = SMALL
    n_prev = {"none_accepted": np.zeros(s.Bt), "all_accepted": np.full(s.Bt, s.k),
              "mixed": np.array([0, 4, 1, 3, 2])}[case].astype(np.int32)
    ver = h.make_verifier(s, kernel)
    lay = h.Layer(s)
    r = synth.Rounds(s, synth.token_stream(s, 0, 32))
    r.cursor, r.n_prev = n_prev.astype(np.int64), n_prev.copy()
    b = r.batch()
    state_before = lay.state.clone()
    conv_before = lay.conv.clone()
    y = lay.gpu_verify(ver, b, s.k)
    lay.check(y, lay.oracle_verify(b, s.k), h.TOL[s.act], case)
    for bi in np.nonzero(n_prev == 0)[0]:   # nothing accepted: the cache is bit-for-bit untouched
        assert torch.equal(lay.state[bi], state_before[bi]) and torch.equal(lay.conv[bi], conv_before[bi])
    assert ver.status() == 0
    ver.close()


@pytest.mark.parametrize("s,kernel", [(SMALL, GENERIC), (SMALL, STREAM), (SMALL64, STREAM), (ODD, GENERIC),
                                      (NOGATE, STREAM), (NOGATE, GENERIC)])
def test_pure_advance_and_odd_shapes(s, kernel):
    """k = 0 folds the pending tokens into the cache and returns their outputs; also covers a
    64-wide state, no gate, and a shape only the generic kernel takes (fp32, W=3, N=40)."""
    h = H()
    ver = h.make_verifier(s, kernel)
    lay = h.Layer(s)
    r = synth.Rounds(s, synth.token_stream(s, 0, 32))
    for rd, (a, k) in enumerate([(None, s.k), (np.arange(s.Bt) % (s.k + 1), s.k), (np.full(s.Bt, s.k), 0),
                                 (np.zeros(s.Bt), 0), (np.zeros(s.Bt), s.k)]):
        if a is not None:
            r.accept(a.astype(np.int32))
        b = r.batch(k=k)
        y = lay.gpu_verify(ver, b, k)
        lay.check(y, lay.oracle_verify(b, k), h.TOL[s.act], f"{s.name} call {rd}")
    assert ver.status() == 0
    ver.close()


@pytest.mark.parametrize("kernel", [GENERIC, STREAM])
def test_out_of_range_n_prev_is_clamped_and_flagged(kernel):
    h = H()
    s = SMALL
    ver = h.make_verifier(s, kernel)
    lay = h.Layer(s)
    r = synth.Rounds(s, synth.token_stream(s, 0, 32))
    r.cursor, r.n_prev = np.full(s.Bt, 4, dtype=np.int64), np.array([4, 0, 4, 0, 4], dtype=np.int32)
    b = r.batch()
    bad = dict(b, n_prev=np.array([9, -3, 4, 0, 4], dtype=np.int32))   # clamps to 4 and 0: same problem as b
    y = lay.gpu_verify(ver, bad, s.k)
    lay.check(y, lay.oracle_verify(b, s.k), h.TOL[s.act], "clamped")
    assert ver.status() == 1
    assert ver.status() == 0      # reading clears it
    ver.close()


def test_commit_records_n_prev_and_clamps_accept_len():
    from paper_2408_15237_b200 import binding
    h = H()
    s = SMALL
    ver = h.make_verifier(s, 0)
    lay = h.Layer(s)
    r = synth.Rounds(s, synth.token_stream(s, 0, 64))
    for rd in range(4):
        b = r.batch()
        y = lay.gpu_verify(ver, b, s.k, n_prev=None)          # pending lengths come from the last commit
        lay.check(y, lay.oracle_verify(b, s.k), h.TOL[s.act], f"commit round {rd}")
        a = synth.acceptance(s, rd)
        ver.commit(h.dev(a, torch.int32))
        assert binding.mamba_spec_get_n_prev(ver.ctx, s.Bt) == list(a)
        r.accept(a)
    assert ver.status() == 0
    ver.commit(h.dev(np.array([7, -1, 2, 0, 4], dtype=np.int32), torch.int32))
    assert binding.mamba_spec_get_n_prev(ver.ctx, s.Bt) == [4, 0, 2, 0, 4]
    assert ver.status() == binding.STATUS_ACCEPT_CLAMPED
    ver.close()


@pytest.mark.parametrize("kernel", [GENERIC, STREAM])
def test_nothing_outside_the_tensors_is_written_and_runs_are_bitwise_repeatable(kernel):
    """Canary words around y, state and conv_state (the sanitizer is not available), rows beyond T_b
    of y keep their contents, and two runs from the same inputs agree bit for bit (no atomics)."""
    h = H()
    s = SMALL
    ad = h.act_dtype(s)
    ver = h.make_verifier(s, kernel)
    r = synth.Rounds(s, synth.token_stream(s, 0, 32))
    r.cursor, r.n_prev = np.full(s.Bt, 4, dtype=np.int64), np.array([1, 0, 4, 2, 3], dtype=np.int32)
    b = r.batch()
    outs = []
    for rep in range(2):
        lay = h.Layer(s)
        guard = 64

        def padded(t, fill):
            buf = torch.full((t.numel() + 2 * guard,), fill, dtype=t.dtype, device="cuda")
            view = buf[guard:guard + t.numel()].view(t.shape)
            view.copy_(t)
            return buf, view
        sbuf, lay.state = padded(lay.state, 7.25)
        cbuf, lay.conv = padded(lay.conv, 7.25)
        ybuf, y = padded(torch.full((s.Bt, s.t_max, s.H, s.P), -3.5, dtype=ad, device="cuda"), 7.25)
        lay.gpu_verify(ver, b, s.k, y=y)
        for buf in (sbuf, cbuf, ybuf):
            assert (buf[:guard] == 7.25).all() and (buf[-guard:] == 7.25).all()
        for bi, j in enumerate(b["n_prev"]):
            assert (y[bi, j + s.k:] == -3.5).all()
            assert not (y[bi, :j + s.k] == -3.5).all()
        outs.append((y.clone(), lay.state.clone(), lay.conv.clone()))
    for a_, b_ in zip(outs[0], outs[1]):
        assert torch.equal(a_, b_)
    ver.close()


def test_generic_and_streaming_kernels_agree():
    h = H()
    s = SMALL
    res = []
    for kernel in (GENERIC, STREAM):
        ver = h.make_verifier(s, kernel)
        lay = h.Layer(s)
        r = synth.Rounds(s, synth.token_stream(s, 0, 32))
        r.cursor, r.n_prev = np.full(s.Bt, 4, dtype=np.int64), np.array([4, 3, 2, 1, 0], dtype=np.int32)
        y = lay.gpu_verify(ver, r.batch(), s.k)
        res.append((y.float().cpu().numpy(), lay.state.cpu().numpy()))
        ver.close()
    valid = ~np.isnan(res[0][0])
    assert np.array_equal(valid, ~np.isnan(res[1][0]))
    assert h.rel_l2(res[0][0][valid], res[1][0][valid]) < 3e-3      # two bf16 roundings apart at most
    assert h.rel_l2(res[0][1], res[1][1]) < 1e-5


def test_host_buffer_entry_point_matches_device_entry_point():
    from paper_2408_15237_b200 import binding
    h = H()
    s = SMALL
    ad = h.act_dtype(s)
    r = synth.Rounds(s, synth.token_stream(s, 0, 32))
    r.cursor, r.n_prev = np.full(s.Bt, 4, dtype=np.int64), np.array([2, 0, 4, 1, 3], dtype=np.int32)
    b = r.batch()
    ver = h.make_verifier(s, 0)
    lay_d, lay_h = h.Layer(s), h.Layer(s)
    y_d = lay_d.gpu_verify(ver, b, s.k)
    host = {n: torch.from_numpy(np.ascontiguousarray(b[n])).to(ad).pin_memory() for n in ("x", "z", "dt", "B", "C")}
    n_prev_h = torch.from_numpy(b["n_prev"]).pin_memory()
    y_h = torch.empty((s.Bt, s.t_max, s.H, s.P), dtype=ad).pin_memory()
    io = binding.IO(lay_h.cw.data_ptr(), lay_h.cb.data_ptr(), host["z"].data_ptr(), y_h.data_ptr(), s.Bt, 0, s.t_max,
                    torch.cuda.current_stream().cuda_stream)
    binding.mamba_spec_verify_host(ver.ctx, lay_h.state, lay_h.conv, host["x"], host["dt"], host["B"], host["C"],
                                   lay_h.A, lay_h.D, n_prev_h, s.k, io)
    torch.cuda.synchronize()
    for bi, j in enumerate(b["n_prev"]):
        assert torch.equal(y_h[bi, :j + s.k], y_d[bi, :j + s.k].cpu())
    assert torch.equal(lay_h.state, lay_d.state) and torch.equal(lay_h.conv, lay_d.conv)
    ver.close()


def test_argument_errors_are_codes_not_crashes():
    from paper_2408_15237_b200 import binding
    h = H()
    s = SMALL
    ver = h.make_verifier(s, 0)
    lay = h.Layer(s)
    ad = h.act_dtype(s)
    x = torch.zeros((s.Bt, s.t_max, s.H, s.P), dtype=ad, device="cuda")
    dt = torch.zeros((s.Bt, s.t_max, s.H), dtype=ad, device="cuda")
    Bm = torch.zeros((s.Bt, s.t_max, s.GB, s.N), dtype=ad, device="cuda")
    Cm = torch.zeros((s.Bt, s.t_max, s.GC, s.N), dtype=ad, device="cuda")
    y = torch.zeros_like(x)

    def call(k=s.k, io_over=None, **over):
        a = dict(state=lay.state, conv=lay.conv, x=x, dt=dt, B=Bm, C=Cm, A=lay.A, D=lay.D)
        a.update(over)
        io = dict(conv_w=lay.cw.data_ptr(), conv_b=lay.cb.data_ptr(), z=x.data_ptr(), y=y.data_ptr(), batch=s.Bt,
                  layer=0, t_max=s.t_max, stream=None)
        io.update(io_over or {})
        ptr = lambda t: None if t is None else (t if isinstance(t, int) else t.data_ptr())
        return binding.lib.mamba_spec_verify(ver.ctx, ptr(a["state"]), ptr(a["conv"]), ptr(a["x"]), ptr(a["dt"]),
                                             ptr(a["B"]), ptr(a["C"]), ptr(a["A"]), ptr(a["D"]), None, k,
                                             ctypes.byref(binding.IO(**io)))
    assert call() == 0
    assert call(x=None) == binding.ERR_INVALID_ARG
    assert call(k=s.k + 1) == binding.ERR_INVALID_ARG
    assert call(k=-1) == binding.ERR_INVALID_ARG
    assert call(io_over=dict(batch=s.Bt + 1)) == binding.ERR_BAD_SHAPE
    assert call(io_over=dict(t_max=s.k - 1)) == binding.ERR_BAD_SHAPE
    assert call(io_over=dict(layer=3)) == binding.ERR_INVALID_ARG
    assert call(io_over=dict(z=None)) == binding.ERR_INVALID_ARG
    assert call(x=x.data_ptr() + 2) == binding.ERR_MISALIGNED
    assert "16-byte" in binding.mamba_spec_last_error(ver.ctx)
    assert binding.lib.mamba_spec_commit(ver.ctx, None, s.Bt, None) == binding.ERR_INVALID_ARG
    torch.cuda.synchronize()
    ver.close()
    # the normalised output needs its weight and a usable eps
    ver = h.make_verifier(synth.replace(s, flags=s.flags | synth.FLAG_GATED_RMSNORM), 0)
    w = torch.ones(s.H * s.P, dtype=torch.float32, device="cuda")
    assert call(io_over=dict(norm_weight=w.data_ptr(), norm_eps=1e-5)) == 0
    assert call() == binding.ERR_INVALID_ARG
    assert call(io_over=dict(norm_weight=w.data_ptr(), norm_eps=-1.0)) == binding.ERR_INVALID_ARG
    assert call(io_over=dict(norm_weight=w.data_ptr(), norm_eps=float("nan"))) == binding.ERR_INVALID_ARG
    torch.cuda.synchronize()
    ver.close()
    odd = synth.Shape("unsup", Bt=1, H=3, P=12, N=40, GB=1, GC=3, W=3, k=2, act="fp32")
    v2 = h.make_verifier(odd, STREAM)          # init succeeds; the launch refuses the shape
    lay2 = h.Layer(odd)
    with pytest.raises(binding.MambaSpecError) as e:
        lay2.gpu_verify(v2, synth.Rounds(odd, synth.token_stream(odd, 0, 8)).batch(), odd.k)
    assert e.value.code == binding.ERR_UNSUPPORTED
    v2.close()


@pytest.mark.parametrize("step,kernel", [(1, STREAM), (2, STREAM), (16, STREAM), (16, GENERIC), (32, GENERIC), (32, STREAM),
                                         (24, STREAM)])
def test_multistep_decoding_from_the_cached_state(step, kernel):
    """The paper's second use of the kernel (Fig. 3): no pending tokens, `step` new tokens per call, t_max = step.
    Three calls in a row; the cache must stay bit-for-bit untouched (nothing was accepted)."""
    h = H()
    s = synth.Shape(f"multistep_{step}", Bt=3, H=8, P=64, N=128, GB=2, GC=8, W=4, k=step, act="bf16", accept="none",
                    t_rows=step)
    ver = h.make_verifier(s, kernel)
    lay = h.Layer(s)
    r = synth.Rounds(s, synth.token_stream(s, 0, 4 * step))
    state_before, conv_before = lay.state.clone(), lay.conv.clone()
    for call in range(3):
        b = r.batch()
        y = lay.gpu_verify(ver, b, s.k)
        lay.check(y, lay.oracle_verify(b, s.k), h.TOL[s.act], f"step {step}, call {call}")
        r.accept(synth.acceptance(s, call))
    assert torch.equal(lay.state, state_before) and torch.equal(lay.conv, conv_before)
    assert ("stream" in ver.last_kernel) == (kernel == STREAM)
    assert ver.status() == 0
    ver.close()


@pytest.mark.parametrize("kernel", [GENERIC, STREAM])
def test_draft_side_step_replays_the_accepted_tokens_and_decodes_one(kernel):
    """The draft model's use of the same call (Sec. 4.3, last paragraph): one launch folds the tokens the
    verifier accepted last round (up to k_max = 4 here) into the cache and decodes one new token: k = 1,
    t_max = 5.  130M-like layer shape (24 heads of 64 channels, state 128)."""
    h = H()
    s = synth.Shape("draft_step", Bt=6, H=24, P=64, N=128, GB=1, GC=1, W=4, k=1, act="bf16", t_rows=5)
    ver = h.make_verifier(s, kernel, k_max=4)
    lay = h.Layer(s)
    r = synth.Rounds(s, synth.token_stream(s, 0, 32))
    for call, n_prev in enumerate([[0, 1, 2, 3, 4, 2], [4, 4, 0, 1, 3, 0]]):
        n_prev = np.asarray(n_prev, dtype=np.int32)
        r.cursor, r.n_prev = r.cursor + n_prev if call else n_prev.astype(np.int64), n_prev.copy()
        b = r.batch()
        y = lay.gpu_verify(ver, b, s.k)
        lay.check(y, lay.oracle_verify(b, s.k), h.TOL[s.act], f"draft step, call {call}")
    assert ("stream" in ver.last_kernel) == (kernel == STREAM)
    assert ver.status() == 0
    ver.close()


LONG = synth.Shape("edge_long", Bt=3, H=8, P=64, N=128, GB=2, GC=8, W=4, k=8, act="bf16")
# 20 new rows on top of up to 8 pending ones: a token block that the streaming kernel takes in segments
BLOCK28 = synth.Shape("edge_block28", Bt=3, H=8, P=64, N=128, GB=2, GC=8, W=4, k=20, act="bf16", t_rows=28, k_prev=8)
# and up to 20 pending ones (40 rows): the pending rows beyond 8 are replayed by launches of their own
BLOCK40 = synth.Shape("edge_block40", Bt=5, H=8, P=64, N=128, GB=2, GC=8, W=4, k=20, act="bf16")


@pytest.mark.parametrize("kernel", [GENERIC, STREAM])
@pytest.mark.parametrize("s", [SMALL, SMALL64, LONG, BLOCK28], ids=["n128", "n64", "k8", "k20"])
def test_second_snapshot_after_all_tokens(s, kernel):
    """MAMBA_SPEC_FLAG_STATE_K (Algorithm 2 caches h_j and h_k): besides the cache at the verified position j
    the call leaves the cache after all T_b = j_b + k tokens in a second pair of buffers.  The oracle for the
    second snapshot is its own pure advance (k = 0) over the T_b rows of the same slab, from the same cache."""
    import oracle
    h = H()
    s2 = synth.replace(s, name=s.name + "_snap2", flags=s.flags | synth.FLAG_STATE_K)
    ver = h.make_verifier(s2, kernel)
    lay = h.Layer(s)
    ad = h.act_dtype(s)
    r = synth.Rounds(s, synth.token_stream(s, 0, 48))
    cap = s.k_prev if s.k_prev else s.k
    pend = [np.arange(s.Bt) % (cap + 1), np.zeros(s.Bt), np.full(s.Bt, cap)]
    for call, n_prev in enumerate(pend):
        n_prev = n_prev.astype(np.int32)
        r.cursor, r.n_prev = (r.cursor + n_prev if call else n_prev.astype(np.int64)), n_prev.copy()
        b = r.batch()
        z = b["z"] if s.flags & synth.FLAG_GATE else None
        _, want_state_k, want_conv_k = oracle.verify(lay.o_state.copy(), lay.o_conv.copy(), b["x"], b["dt"], b["B"], b["C"],
                                                     lay.np["A"], lay.np["D"], lay.np["cw"], lay.np["cb"], z,
                                                     (n_prev + s.k).astype(np.int32), 0, s.flags)
        y_ref = lay.oracle_verify(b, s.k)
        t = {n: h.dev(b[n], ad) for n in ("x", "z", "dt", "B", "C")}
        y = torch.full(t["x"].shape, float("nan"), device="cuda", dtype=ad)
        state_k = torch.full_like(lay.state, float("nan"))
        conv_k = torch.full_like(lay.conv, float("nan"))
        ver.verify(lay.state, lay.conv, t["x"], t["dt"], t["B"], t["C"], lay.A, lay.D, lay.cw, lay.cb,
                   t["z"] if s.flags & synth.FLAG_GATE else None, y, h.dev(b["n_prev"], torch.int32), s.k,
                   state_k=state_k, conv_state_k=conv_k)
        torch.cuda.synchronize()
        lay.check(y, y_ref, h.TOL[s.act], f"second snapshot, call {call}")      # y and the cache at position j
        assert h.rel_l2(state_k.cpu().numpy(), want_state_k) <= h.TOL["fp32"], f"call {call}: state after all tokens"
        assert np.array_equal(conv_k.float().cpu().numpy().astype(np.float64), want_conv_k), f"call {call}: conv window after all tokens"
    assert ("stream" in ver.last_kernel) == (kernel == STREAM)
    assert ver.status() == 0
    ver.close()


@pytest.mark.parametrize("kernel", [GENERIC, STREAM])
def test_checkpoint_and_resume_in_a_fresh_context(kernel):
    """A decoder's whole resumable state per layer is the cached state, the conv window and the pending lengths
    (Sec. 4.2; Sec. 4.3, footnote).  After round 3 these are saved, the context is destroyed, a fresh context
    and fresh device buffers are loaded from the copy, and rounds 4..7 must come out bit for bit as in the run
    that was never interrupted."""
    h = H()
    from paper_2408_15237_b200 import binding
    s = synth.SWEEP[(4, 4)]
    ad = h.act_dtype(s)
    stream = synth.token_stream(s, 0, 8 * s.k + s.k + 1)
    acc = [synth.acceptance(s, rd) for rd in range(8)]

    def run(ver, lay, r, rounds):
        outs = []
        for rd in rounds:
            b = r.batch()
            t = {n: h.dev(b[n], ad) for n in ("x", "z", "dt", "B", "C")}
            y = torch.full(t["x"].shape, float("nan"), device="cuda", dtype=ad)
            ver.verify(lay.state, lay.conv, t["x"], t["dt"], t["B"], t["C"], lay.A, lay.D, lay.cw, lay.cb, t["z"], y, None, s.k)
            ver.commit(h.dev(acc[rd], torch.int32))
            torch.cuda.synchronize()
            outs.append(y.clone())
            r.accept(acc[rd])
        return outs

    # the uninterrupted run
    ver_a, lay_a, r_a = h.make_verifier(s, kernel), h.Layer(s), synth.Rounds(s, stream)
    run(ver_a, lay_a, r_a, range(4))
    saved = dict(state=lay_a.state.cpu().clone(), conv=lay_a.conv.cpu().clone(), n_prev=binding.mamba_spec_get_n_prev(ver_a.ctx, s.Bt),
                 cursor=r_a.cursor.copy())
    want = run(ver_a, lay_a, r_a, range(4, 8))
    want_state, want_conv = lay_a.state.clone(), lay_a.conv.clone()
    ver_a.close()
    # the resumed run: fresh context, fresh buffers, pending lengths handed back through commit
    ver_b, lay_b, r_b = h.make_verifier(s, kernel), h.Layer(s), synth.Rounds(s, stream)
    lay_b.state.copy_(saved["state"])
    lay_b.conv.copy_(saved["conv"])
    assert saved["n_prev"] == [int(v) for v in acc[3]]
    # (a fresh context has no pending lengths yet: the saved ones go back in through commit, which clamps to the
    #  draft length of the last verify, or to k_max when there has been none)
    binding.lib.mamba_spec_commit(ver_b.ctx, h.dev(np.asarray(saved["n_prev"], dtype=np.int32), torch.int32).data_ptr(), s.Bt,
                                  torch.cuda.current_stream().cuda_stream)
    r_b.cursor, r_b.n_prev = saved["cursor"].copy(), np.asarray(saved["n_prev"], dtype=np.int32)
    got = run(ver_b, lay_b, r_b, range(4, 8))
    for a, b_ in zip(want, got):
        assert torch.equal(torch.nan_to_num(a.float(), nan=-7.0), torch.nan_to_num(b_.float(), nan=-7.0))
    assert torch.equal(lay_b.state, want_state) and torch.equal(lay_b.conv, want_conv)
    assert ver_b.status() == 0
    ver_b.close()


@pytest.mark.parametrize("kernel", [GENERIC, STREAM])
@pytest.mark.parametrize("s", [BLOCK28, BLOCK40], ids=["pending8", "pending20"])
def test_token_blocks_longer_than_sixteen_rows_with_pending_tokens(s, kernel):
    """20 new tokens per call on top of up to 8 (28 rows) or up to 20 (40 rows) pending ones: the streaming
    kernel takes such a block in launches of at most 16 rows with at most 8 pending ones, carrying the state from
    one to the next; outputs in float32 so that the bound is the arithmetic's 1e-5.  Four rounds with mixed
    acceptance, then a call with no drafts that only replays the pending rows."""
    h = H()
    worst, name = h.run_rounds(s, 4, kernel=kernel, first_j=5, y_f32=True, tol=1e-5, final_flush=True)
    assert ("stream" in name) == (kernel == STREAM)
    assert max(worst) <= 1e-5
