"""GPU parity of the parameterisation variants against the fp64 oracle, through the C ABI:
the Mamba-1 form (Algorithm 1), the softplus of a raw interval taken in the kernel (Sec. 2.2), and
Algorithm 2's choice between h_j and h_k made by commit (two buffers per sequence, no replay after a
fully accepted round)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2408_15237_b200 import synth

pytestmark = pytest.mark.gpu

GENERIC, STREAM = 1, 2


def H():
    import harness
    return harness


M1_SMALL = synth.Shape("m1_small", Bt=3, H=4, P=16, N=32, GB=2, GC=4, W=4, k=3, act="fp32")
M1_BF16 = synth.Shape("m1_bf16", Bt=2, H=8, P=64, N=128, GB=2, GC=8, W=4, k=4, act="bf16")


@pytest.mark.parametrize("s,tol", [(M1_SMALL, 1e-5), (M1_BF16, 1e-5)])
def test_mamba1_form_matches_the_oracle(s, tol):
    """Interval per channel, A per (channel, state column), D per channel; y in float32 so that the only error
    left is the kernel's fp32 arithmetic.  Three rounds with replay, then a flush."""
    h = H()
    from paper_2408_15237_b200 import binding
    flags = s.flags | binding.FLAG_MAMBA1 | binding.FLAG_Y_F32
    ver = binding.Verifier(s.Bt, s.H, s.P, s.N, s.GB, s.GC, s.W, s.k, act=s.act, flags=flags)
    ad = h.act_dtype(s)
    A, D = synth.m1_params(s)
    _, _, cw, cb = synth.layer_params(s)
    st, cv = synth.initial_cache(s)
    L = 4 * s.k + 4
    stream = synth.token_stream(s, 0, L)
    stream["dt"] = synth.m1_dt_stream(s, 0, L)
    r = synth.Rounds(s, stream, first_j=2)
    o_state, o_conv = st.astype(np.float64), cv.astype(np.float64)
    state, conv = h.dev(st, torch.float32), h.dev(cv, ad)
    dA, dD, dcw, dcb = (h.dev(a, torch.float32) for a in (A, D, cw, cb))
    for rd, k in enumerate([s.k, s.k, s.k, 0]):
        b = r.batch(k=k)
        t = {n: h.dev(b[n], ad) for n in ("x", "z", "dt", "B", "C")}
        y = torch.full(t["x"].shape, float("nan"), device="cuda", dtype=torch.float32)
        ver.verify(state, conv, t["x"], t["dt"], t["B"], t["C"], dA, dD, dcw, dcb, t["z"], y, h.dev(b["n_prev"], torch.int32), k)
        torch.cuda.synchronize()
        assert ver.last_kernel == "generic"
        y_ref, o_state, o_conv = oracle.verify_m1(o_state, o_conv, b["x"], b["dt"], b["B"], b["C"], A, D, cw, cb, b["z"],
                                                   b["n_prev"], k, s.flags, threads=oracle.host_threads())
        yg = y.cpu().numpy().astype(np.float64)
        valid = ~np.isnan(y_ref)
        assert np.isnan(yg[~valid]).all() and not np.isnan(yg[valid]).any()
        if valid.any():
            assert h.rel_l2(yg[valid], y_ref[valid]) <= tol, f"round {rd}"
        assert h.rel_l2(state.cpu().numpy(), o_state) <= tol, f"round {rd}"
        assert np.abs(conv.float().cpu().numpy().astype(np.float64) - o_conv).max() == 0.0
        if k:
            r.accept(synth.acceptance(s, rd))
    assert ver.status() == 0
    ver.close()


@pytest.mark.parametrize("s,kernel,m1", [(synth.CONFIGS[0], GENERIC, False), (M1_SMALL, GENERIC, True),
                                         (synth.SWEEP[(4, 4)], STREAM, False), (synth.SWEEP[(4, 4)], GENERIC, False)])
def test_softplus_of_the_raw_interval_in_the_kernel(s, kernel, m1):
    """dt arrives raw with a bias; the kernel's softplus(dt + bias) against the oracle fed with the interval
    computed on the host in fp64."""
    h = H()
    from paper_2408_15237_b200 import binding
    flags = s.flags | binding.FLAG_DT_SOFTPLUS | binding.FLAG_Y_F32 | (binding.FLAG_MAMBA1 if m1 else 0)
    ver = binding.Verifier(s.Bt, s.H, s.P, s.N, s.GB, s.GC, s.W, s.k, act=s.act, flags=flags, kernel=kernel)
    ad = h.act_dtype(s)
    A, D, cw, cb = synth.layer_params(s)
    if m1:
        A, D = synth.m1_params(s)
    st, cv = synth.initial_cache(s)
    L = 3 * s.k + 4
    stream = synth.token_stream(s, 0, L)
    raw, bias = synth.raw_dt_stream(s, 0, L, per_channel=m1)
    stream["dt"] = raw
    r = synth.Rounds(s, stream, first_j=min(2, s.k))
    o_state, o_conv = st.astype(np.float64), cv.astype(np.float64)
    state, conv = h.dev(st, torch.float32), h.dev(cv, ad)
    dA, dD, dcw, dcb, dbias = (h.dev(a, torch.float32) for a in (A, D, cw, cb, bias))
    for rd in range(3):
        b = r.batch()
        t = {n: h.dev(b[n], ad) for n in ("x", "z", "dt", "B", "C")}
        y = torch.full(t["x"].shape, float("nan"), device="cuda", dtype=torch.float32)
        ver.verify(state, conv, t["x"], t["dt"], t["B"], t["C"], dA, dD, dcw, dcb, t["z"], y, h.dev(b["n_prev"], torch.int32),
                   s.k, dt_bias=dbias)
        torch.cuda.synchronize()
        assert ("stream" in ver.last_kernel) == (kernel == STREAM)
        dt_eff = oracle.softplus_dt(np.nan_to_num(b["dt"]), bias)
        fn = oracle.verify_m1 if m1 else oracle.verify
        y_ref, o_state, o_conv = fn(o_state, o_conv, b["x"], dt_eff, b["B"], b["C"], A, D, cw, cb, b["z"], b["n_prev"], s.k,
                                    s.flags, threads=oracle.host_threads())
        yg = y.cpu().numpy().astype(np.float64)
        valid = ~np.isnan(y_ref)
        assert np.isnan(yg[~valid]).all() and not np.isnan(yg[valid]).any()
        assert h.rel_l2(yg[valid], y_ref[valid]) <= 1e-5, f"round {rd}"
        assert h.rel_l2(state.cpu().numpy(), o_state) <= 1e-5, f"round {rd}"
        r.accept(synth.acceptance(s, rd))
    assert ver.status() == 0
    ver.close()


@pytest.mark.parametrize("s,kernel", [(synth.CONFIGS[0], GENERIC), (synth.SWEEP[(4, 4)], STREAM), (synth.SWEEP[(4, 4)], GENERIC),
                                      (synth.CONFIGS[3], STREAM)])
def test_commit_selects_h_k_after_a_fully_accepted_round(s, kernel):
    """Algorithm 2: a round whose drafts were all accepted keeps h_k, any other keeps h_j and replays.  Eight
    rounds with a mix of full and partial acceptance through verify + commit on two buffers per sequence; the
    returned rows and, at the end, each sequence's cache (wherever commit left it) against the oracle's plain
    sequential run over the accepted tokens."""
    h = H()
    from paper_2408_15237_b200 import binding
    flags = s.flags | binding.FLAG_STATE_K | binding.FLAG_COMMIT_SELECTS | binding.FLAG_Y_F32
    ver = binding.Verifier(s.Bt, s.H, s.P, s.N, s.GB, s.GC, s.W, s.k, act=s.act, flags=flags, kernel=kernel)
    ad = h.act_dtype(s)
    A, D, cw, cb = synth.layer_params(s)
    st, cv = synth.initial_cache(s)
    rounds = 8
    L = rounds * s.k + s.k + 1
    stream = synth.token_stream(s, 0, L)
    r = synth.Rounds(s, stream, first_j=0)
    bufs = [(h.dev(st, torch.float32), h.dev(cv, ad)), (torch.full_like(h.dev(st, torch.float32), float("nan")),
                                                        torch.zeros_like(h.dev(cv, ad)))]
    dA, dD, dcw, dcb = (h.dev(a, torch.float32) for a in (A, D, cw, cb))
    y_seq, st_seq, cv_seq = None, None, None
    g = np.random.default_rng(7)
    total = np.zeros(s.Bt, dtype=np.int64)
    got_rows = {}
    for rd in range(rounds):
        b = r.batch()
        t = {n: h.dev(b[n], ad) for n in ("x", "z", "dt", "B", "C")}
        y = torch.full(t["x"].shape, float("nan"), device="cuda", dtype=torch.float32)
        ver.verify(bufs[0][0], bufs[0][1], t["x"], t["dt"], t["B"], t["C"], dA, dD, dcw, dcb, t["z"], y, None, s.k,
                   state_k=bufs[1][0], conv_state_k=bufs[1][1])
        torch.cuda.synchronize()
        assert ("stream" in ver.last_kernel) == (kernel == STREAM)
        # the pending lengths the library used must be what this bookkeeping expects
        assert ver_n_prev(ver, s.Bt) == [int(v) for v in b["n_prev"]]
        yg = y.cpu().numpy().astype(np.float64)
        rows = r.rows()
        for bi in range(s.Bt):
            for ti in range(rows.shape[1]):
                if rows[bi, ti] >= 0:
                    got_rows[(bi, int(rows[bi, ti]))] = yg[bi, ti]
        # a mix: about half of the sequences accept everything, the others a random prefix
        a = np.where(g.random(s.Bt) < 0.5, s.k, g.integers(0, s.k + 1, s.Bt)).astype(np.int32)
        ver.commit(h.dev(a, torch.int32))
        total += a
        # the harness's bookkeeping of what is pending: nothing after a full acceptance
        r.cursor = r.cursor + a
        r.n_prev = np.where(a == s.k, 0, a).astype(np.int32)
    torch.cuda.synchronize()
    sel = ver.selection(s.Bt)
    # a last flush folds what is still pending into the caches
    b = r.batch(k=0)
    t = {n: h.dev(np.nan_to_num(b[n]), ad) for n in ("x", "z", "dt", "B", "C")}
    y = torch.full(t["x"].shape, float("nan"), device="cuda", dtype=torch.float32)
    ver.verify(bufs[0][0], bufs[0][1], t["x"], t["dt"], t["B"], t["C"], dA, dD, dcw, dcb, t["z"], y, None, 0,
               state_k=bufs[1][0], conv_state_k=bufs[1][1])
    torch.cuda.synchronize()
    assert ver.status() == 0
    y_seq, st_seq, cv_seq = oracle.sequential(st, cv, stream["x"], stream["dt"], stream["B"], stream["C"], A, D, cw, cb,
                                              stream["z"], total.astype(np.int32), s.flags, threads=oracle.host_threads())
    for bi in range(s.Bt):
        cur = bufs[sel[bi]]
        assert h.rel_l2(cur[0][bi].cpu().numpy(), st_seq[bi]) <= 1e-5, f"sequence {bi}: cache"
        assert np.abs(cur[1][bi].float().cpu().numpy().astype(np.float64) - cv_seq[bi]).max() == 0.0, f"sequence {bi}: window"
    # every returned row of an accepted position equals the sequential run's row there
    for (bi, pos), row in got_rows.items():
        if pos < total[bi]:
            assert h.rel_l2(row, y_seq[bi, pos]) <= 1e-5, (bi, pos)
    ver.close()


def ver_n_prev(ver, batch):
    from paper_2408_15237_b200 import binding
    return binding.mamba_spec_get_n_prev(ver.ctx, batch)


@pytest.mark.parametrize("s,kernel,selects,norm", [(synth.CONFIGS[0], GENERIC, False, False), (synth.SWEEP[(4, 4)], STREAM, False, False),
                                              (synth.SWEEP[(4, 4)], STREAM, True, False), (synth.SWEEP[(4, 4)], GENERIC, True, False),
                                              (synth.CONFIGS[3], STREAM, True, False), (synth.SWEEP[(4, 4)], STREAM, False, True),
                                              (synth.SWEEP[(4, 4)], GENERIC, True, True)])
def test_new_rows_only_with_the_library_side_row_store(s, kernel, selects, norm):
    """The caller hands over only the k new rows per round (Sec. 4.2 "caching older entries"); the tokens accepted
    since the last call are replayed from the rows the library kept.  Two layers share the context (each has
    its own kept rows).  Mixed full and partial acceptance over eight rounds; returned rows, final caches and
    conv windows against the oracle's plain sequential run."""
    h = H()
    from paper_2408_15237_b200 import binding
    n_layers = 2
    flags = s.flags | binding.FLAG_Y_F32 | ((binding.FLAG_STATE_K | binding.FLAG_COMMIT_SELECTS) if selects else 0)
    flags |= binding.FLAG_GATED_RMSNORM if norm else 0      # (the normalising kernel then works on [batch][k] rows)
    nw, neps = synth.norm_params(s, 0)
    nkw = dict(norm_weight=h.dev(nw, torch.float32), norm_eps=neps) if norm else {}
    ver = binding.Verifier(s.Bt, s.H, s.P, s.N, s.GB, s.GC, s.W, s.k, act=s.act, flags=flags, kernel=kernel, n_layers=n_layers)
    ad = h.act_dtype(s)
    rounds = 8
    L = rounds * s.k + 1
    lay = []
    for l in range(n_layers):
        A, D, cw, cb = synth.layer_params(s, l)
        st, cv = synth.initial_cache(s, l)
        stream = synth.token_stream(s, l, L)
        bufs = [(h.dev(st, torch.float32), h.dev(cv, ad)),
                (torch.full_like(h.dev(st, torch.float32), float("nan")), torch.zeros_like(h.dev(cv, ad)))]
        lay.append(dict(np=(A, D, cw, cb, st, cv), stream=stream, bufs=bufs, got={},
                        dev=tuple(h.dev(a, torch.float32) for a in (A, D, cw, cb))))
    g = np.random.default_rng(11)
    cursor = np.zeros(s.Bt, dtype=np.int64)     # tokens verified so far
    for rd in range(rounds):
        for l, q in enumerate(lay):
            idx = cursor[:, None] + np.arange(s.k)[None, :]
            bi = np.arange(s.Bt)[:, None]
            t = {n: h.dev(q["stream"][n][bi, idx], ad) for n in ("x", "z", "dt", "B", "C")}
            y = torch.full((s.Bt, s.k, s.H, s.P), float("nan"), device="cuda", dtype=torch.float32)
            dA, dD, dcw, dcb = q["dev"]
            ver.verify_new(q["bufs"][0][0], q["bufs"][0][1], t["x"], t["dt"], t["B"], t["C"], dA, dD, dcw, dcb, t["z"], y, s.k,
                           layer=l, state_k=q["bufs"][1][0] if selects else None, conv_state_k=q["bufs"][1][1] if selects else None, **nkw)
            torch.cuda.synchronize()
            assert ("stream" in ver.last_kernel) == (kernel == STREAM)
            yg = y.cpu().numpy().astype(np.float64)
            for b in range(s.Bt):
                for i in range(s.k):
                    q["got"][(b, int(cursor[b] + i))] = yg[b, i]
        a = np.where(g.random(s.Bt) < 0.4, s.k, g.integers(0, s.k + 1, s.Bt)).astype(np.int32)
        ver.commit(h.dev(a, torch.int32))
        cursor += a
    # flush what is pending
    for l, q in enumerate(lay):
        dA, dD, dcw, dcb = q["dev"]
        y = torch.zeros((s.Bt, 1, s.H, s.P), device="cuda", dtype=torch.float32)
        ver.verify_new(q["bufs"][0][0], q["bufs"][0][1], None, None, None, None, dA, dD, dcw, dcb, None, y, 0, layer=l,
                       state_k=q["bufs"][1][0] if selects else None, conv_state_k=q["bufs"][1][1] if selects else None, **nkw)
    torch.cuda.synchronize()
    assert ver.status() == 0
    sel = ver.selection(s.Bt) if selects else [0] * s.Bt
    for l, q in enumerate(lay):
        A, D, cw, cb, st, cv = q["np"]
        y_seq, st_seq, cv_seq = oracle.sequential(st, cv, q["stream"]["x"], q["stream"]["dt"], q["stream"]["B"], q["stream"]["C"],
                                                  A, D, cw, cb, q["stream"]["z"], cursor.astype(np.int32), s.flags,
                                                  threads=oracle.host_threads())
        if norm:
            y_seq = oracle.gated_rmsnorm(y_seq, nw, neps)
        for b in range(s.Bt):
            cur = q["bufs"][sel[b]]
            assert h.rel_l2(cur[0][b].cpu().numpy(), st_seq[b]) <= 1e-5, f"layer {l} sequence {b}: cache"
            assert np.abs(cur[1][b].float().cpu().numpy().astype(np.float64) - cv_seq[b]).max() == 0.0
        for (b, pos), row in q["got"].items():
            if pos < cursor[b]:
                assert not np.isnan(row).any()
                assert h.rel_l2(row, y_seq[b, pos]) <= 1e-5, (l, b, pos)
    ver.close()


# ------------------------------------------------------------------ gated RMSNorm of the output rows
NORM_SHAPES = [
    synth.Shape("norm_small", Bt=3, H=8, P=64, N=128, GB=2, GC=8, W=4, k=4, act="bf16",
                flags=synth.FLAG_GATE | synth.FLAG_CONV_SILU | synth.FLAG_GATED_RMSNORM),
    synth.replace(synth.llama8b_layer("norm_llama8b_b4", 4, 4), flags=synth.FLAG_GATE | synth.FLAG_CONV_SILU | synth.FLAG_GATED_RMSNORM),
    synth.Shape("norm_fp32", Bt=2, H=2, P=16, N=16, GB=1, GC=2, W=4, k=3, act="fp32",
                flags=synth.FLAG_GATE | synth.FLAG_CONV_SILU | synth.FLAG_GATED_RMSNORM),
]


@pytest.mark.parametrize("kernel", [GENERIC, STREAM])
@pytest.mark.parametrize("s", NORM_SHAPES, ids=lambda s: s.name)
@pytest.mark.parametrize("y_f32", [False, True])
def test_gated_rmsnorm_of_the_output_rows(s, kernel, y_f32):
    """MAMBA_SPEC_FLAG_GATED_RMSNORM: every output row leaves the call normalised over its H*P channels and weighted
    (the oracle applies its own gated_rmsnorm to its own outputs); rows beyond T_b stay untouched; the cache is the
    same as without the flag.  With float32 outputs the bound is 1e-5."""
    if kernel == STREAM and s.act != "bf16":
        pytest.skip("the streaming kernel takes bf16 activations")
    h = H()
    tol = 1e-5 if (y_f32 or s.act == "fp32") else None
    worst, name = h.run_rounds(s, 3, kernel=kernel, first_j=2, y_f32=y_f32, tol=tol, final_flush=True)
    assert ("stream" in name) == (kernel == STREAM)
    if tol:
        assert max(worst) <= tol


# ------------------------------------------------------------------ conv over the B and C channels
BC_FLAGS = synth.FLAG_GATE | synth.FLAG_CONV_SILU | synth.FLAG_CONV_BC
BC_SHAPES = [
    synth.Shape("bc_small_fp32", Bt=3, H=4, P=16, N=32, GB=2, GC=4, W=4, k=3, act="fp32", flags=BC_FLAGS),
    synth.Shape("bc_bf16", Bt=2, H=8, P=64, N=128, GB=2, GC=8, W=4, k=4, act="bf16", flags=BC_FLAGS),
    synth.Shape("bc_w3_norm", Bt=2, H=4, P=32, N=64, GB=1, GC=2, W=3, k=2, act="bf16", flags=BC_FLAGS | synth.FLAG_GATED_RMSNORM),
]


@pytest.mark.parametrize("s", BC_SHAPES, ids=lambda s: s.name)
def test_conv_over_the_b_and_c_channels(s):
    """MAMBA_SPEC_FLAG_CONV_BC: the B and C rows pass through their own rolling conv and activation before the
    recurrence (oracle: verify_conv_bc); y in float32 so that the bound is 1e-5; the window of that conv is cached at
    the verified position exactly.  Four rounds with replay, then a call without drafts."""
    h = H()
    worst, name = h.run_rounds(s, 4, kernel=0, first_j=2, y_f32=True, tol=1e-5, final_flush=True)
    assert name == "generic"
    assert max(worst) <= 1e-5


def test_conv_over_b_and_c_is_refused_where_it_cannot_run():
    from paper_2408_15237_b200 import binding
    s = BC_SHAPES[1]
    with pytest.raises(binding.MambaSpecError):      # the streaming kernel does not take it
        H().make_verifier(s, STREAM)
    with pytest.raises(binding.MambaSpecError):      # one window of B and C rows: no second snapshot
        H().make_verifier(synth.replace(s, flags=s.flags | synth.FLAG_STATE_K), 0)
