"""Pins for the fp64 oracle: each test checks it against something other than itself.

The paper prints no worked numeric example of the kernel, so the pins are what
its equations fix: the multi-step call must equal repeated single steps
(Sec. 4.2), accept-then-advance must equal a direct sequential run (Alg. 2),
and special parameter choices reduce the recurrence (Eq. 1, Sec. 2.2) to closed
forms or to library routines (a cumulative sum, a causal matmul = linearised
attention of Sec. 2.1, numpy's full correlation).
"""
import numpy as np
import pytest

import oracle
from paper_2408_15237_b200 import synth

GATE, CSILU = oracle.FLAG_GATE, oracle.FLAG_CONV_SILU


def small_problem(seed, Bt=3, H=4, P=5, N=6, GB=2, GC=4, W=4, T=7):
    g = np.random.default_rng(seed)
    return dict(
        state=0.3 * g.standard_normal((Bt, H, P, N)),
        conv=0.5 * g.standard_normal((Bt, W - 1, H * P)),
        x=g.standard_normal((Bt, T, H, P)),
        z=g.standard_normal((Bt, T, H, P)),
        dt=np.log1p(np.exp(g.standard_normal((Bt, T, H)) - 1.0)),
        B=g.standard_normal((Bt, T, GB, N)),
        C=g.standard_normal((Bt, T, GC, N)),
        A=-np.exp(g.uniform(0, np.log(16), H)),
        D=g.standard_normal(H),
        cw=g.standard_normal((H * P, W)) / 2,
        cb=0.1 * g.standard_normal(H * P),
    )


def run_verify(q, n_prev, k, flags, **over):
    a = dict(q, **over)
    return oracle.verify(a["state"], a["conv"], a["x"], a["dt"], a["B"], a["C"], a["A"], a["D"],
                         a["cw"], a["cb"], a["z"], n_prev, k, flags)


def full_conv_channels(q, b, flags):
    """Post-conv x of sequence b over the whole stream via numpy's correlate on history ++ stream: [T, H*P]."""
    T = q["x"].shape[1]
    C = q["cw"].shape[0]
    W = q["cw"].shape[1]
    xs = q["x"][b].reshape(T, C)
    out = np.empty((T, C))
    for c in range(C):
        seq = np.concatenate([q["conv"][b, :, c], xs[:, c]])
        v = np.correlate(seq, q["cw"][c], mode="valid") + q["cb"][c]     # length T
        assert v.shape == (T,) and W == q["conv"].shape[1] + 1
        out[:, c] = v / (1 + np.exp(-v)) if flags & CSILU else v
    return out


# --------------------------------------------------------------------------- multi-step == single steps
@pytest.mark.parametrize("flags", [0, GATE, CSILU, GATE | CSILU])
def test_multistep_equals_repeated_single_steps(flags):
    q = small_problem(1)
    Bt, T = q["x"].shape[:2]
    k = 3
    n_prev = np.array([4, 0, 2], dtype=np.int32)
    y, s_out, c_out = run_verify(q, n_prev, k, flags)
    st, cv = q["state"].copy(), q["conv"].copy()
    snap_s, snap_c = st.copy(), cv.copy()
    for t in range(T):
        active = (t < n_prev + k).astype(np.int32)
        y1, st, cv = oracle.step(st, cv, q["x"][:, t], q["dt"][:, t], q["B"][:, t], q["C"][:, t], q["A"], q["D"],
                                 q["cw"], q["cb"], q["z"][:, t], flags, active)
        for b in range(Bt):
            if active[b]:
                np.testing.assert_allclose(y[b, t], y1[b], rtol=1e-12, atol=1e-13)
            else:
                assert np.isnan(y[b, t]).all()
            if t == n_prev[b] - 1:
                snap_s[b], snap_c[b] = st[b], cv[b]
    np.testing.assert_allclose(s_out, snap_s, rtol=1e-12, atol=1e-14)
    np.testing.assert_array_equal(c_out, snap_c)
    # the sequence with nothing accepted keeps its cache bit for bit
    np.testing.assert_array_equal(s_out[1], q["state"][1])
    np.testing.assert_array_equal(c_out[1], q["conv"][1])


# --------------------------------------------------------------------------- accept-then-advance == sequential
@pytest.mark.parametrize("cfg", [0, "geo"])
def test_speculation_rounds_equal_direct_sequential_run(cfg):
    if cfg == 0:
        s = synth.CONFIGS[0]
    else:
        s = synth.Shape("pin_geo", Bt=3, H=4, P=8, N=4, GB=2, GC=4, W=4, k=3, act="bf16",
                        accept="geometric", accept_p=0.4, rounds=12)
    A, D, cw, cb = synth.layer_params(s)
    st0, cv0 = synth.initial_cache(s)
    stream = synth.token_stream(s, 0, s.rounds * s.k + s.k + s.first_j + 1)
    r = synth.Rounds(s, stream, first_j=s.first_j)
    st, cv = st0.astype(np.float64), cv0.astype(np.float64)
    seen = []
    for rd in range(s.rounds):
        b = r.batch()
        rows = r.rows()
        y, st, cv = oracle.verify(st, cv, b["x"], b["dt"], b["B"], b["C"], A, D, cw, cb, b["z"], b["n_prev"],
                                  s.k, s.flags)
        seen.append((rows, y))
        r.accept(synth.acceptance(s, rd))
    # final flush: k = 0 folds the last accepted tokens into the cache
    b = r.batch()
    _, st, cv = oracle.verify(st, cv, b["x"], b["dt"], b["B"], b["C"], A, D, cw, cb, b["z"], b["n_prev"], 0, s.flags)

    L = stream["x"].shape[1]
    y_seq_all, _, _ = oracle.sequential(st0, cv0, stream["x"], stream["dt"], stream["B"], stream["C"], A, D, cw, cb,
                                        stream["z"], np.full(s.Bt, L), s.flags)
    _, st_seq, cv_seq = oracle.sequential(st0, cv0, stream["x"], stream["dt"], stream["B"], stream["C"], A, D, cw,
                                          cb, stream["z"], r.cursor, s.flags)
    assert r.cursor.max() > s.k            # the run really advanced
    np.testing.assert_allclose(st, st_seq, rtol=1e-12, atol=1e-14)
    np.testing.assert_array_equal(cv, cv_seq)
    for rows, y in seen:                   # every returned row is the stream's output at that position
        for bi in range(s.Bt):
            for t, row in enumerate(rows[bi]):
                if row >= 0:
                    np.testing.assert_allclose(y[bi, t], y_seq_all[bi, row], rtol=1e-11, atol=1e-13)
                else:
                    assert np.isnan(y[bi, t]).all()


# --------------------------------------------------------------------------- closed forms
def test_dt_zero_leaves_state_and_gives_C_h0_plus_D_xc():
    q = small_problem(2)
    n_prev = np.array([3, 1, 4], dtype=np.int32)
    k, flags = 3, CSILU
    y, s_out, _ = run_verify(q, n_prev, k, flags, dt=np.zeros_like(q["dt"]))
    np.testing.assert_array_equal(s_out, q["state"])
    Bt, T, H, P = q["x"].shape
    for b in range(Bt):
        xc = full_conv_channels(q, b, flags).reshape(T, H, P)
        for t in range(n_prev[b] + k):
            for h in range(H):
                want = q["state"][b, h] @ q["C"][b, t, h // (H // q["C"].shape[2])] + q["D"][h] * xc[t, h]
                np.testing.assert_allclose(y[b, t, h], want, rtol=1e-12, atol=1e-13)


def test_zero_input_matrix_gives_pure_exponential_decay():
    q = small_problem(3)
    n_prev = np.array([4, 2, 3], dtype=np.int32)
    dt = np.full_like(q["dt"], 0.37)
    y, s_out, _ = run_verify(q, n_prev, 2, GATE | CSILU, B=np.zeros_like(q["B"]), dt=dt)
    for b, j in enumerate(n_prev):
        want = q["state"][b] * np.exp(q["A"] * 0.37 * j)[:, None, None]
        np.testing.assert_allclose(s_out[b], want, rtol=1e-13)


def test_A_to_zero_gives_cumulative_sum_of_rank_one_updates():
    q = small_problem(4)
    Bt, T, H, P = q["x"].shape
    n_prev = np.array([4, 3, 1], dtype=np.int32)
    flags = CSILU
    y, s_out, _ = run_verify(q, n_prev, 3, flags, A=np.zeros_like(q["A"]))
    GB = q["B"].shape[2]
    for b, j in enumerate(n_prev):
        xc = full_conv_channels(q, b, flags).reshape(T, H, P)
        for h in range(H):
            upd = [q["dt"][b, t, h] * np.outer(xc[t, h], q["B"][b, t, h // (H // GB)]) for t in range(j)]
            want = q["state"][b, h] + np.cumsum(np.stack(upd), axis=0)[-1]
            np.testing.assert_allclose(s_out[b, h], want, rtol=1e-12, atol=1e-14)


def test_linearised_attention_special_case_is_a_causal_matmul():
    """A=0 (decay 1), dt=1, h0=0, D=0, identity conv: y = tril(C B^T) x, the linear-attention form of Sec. 2.1."""
    q = small_problem(5, Bt=2, H=4, P=3, N=5, GB=2, GC=1, T=6)
    Bt, T, H, P = q["x"].shape
    cw = np.zeros_like(q["cw"])
    cw[:, -1] = 1.0
    y, s_out, _ = run_verify(q, np.array([2, 0], dtype=np.int32), 4, 0, A=np.zeros(H), D=np.zeros(H),
                             dt=np.ones_like(q["dt"]), state=np.zeros_like(q["state"]), cw=cw,
                             cb=np.zeros_like(q["cb"]))
    for b, Tb in enumerate([6, 4]):
        for h in range(H):
            Q, K, V = q["C"][b, :Tb, 0], q["B"][b, :Tb, h // 2], q["x"][b, :Tb, h]
            want = np.tril(Q @ K.T) @ V
            np.testing.assert_allclose(y[b, :Tb, h], want, rtol=1e-12, atol=1e-13)
    # state after the 2 replayed tokens of sequence 0: sum_s x_s B_s^T
    for h in range(H):
        want = sum(np.outer(q["x"][0, s_, h], q["B"][0, s_, h // 2]) for s_ in range(2))
        np.testing.assert_allclose(s_out[0, h], want, rtol=1e-12, atol=1e-14)


def test_brute_force_unrolled_sums_on_tiny_input():
    """y_t and h_j written as explicit sums over earlier tokens, with no recurrence at all."""
    q = small_problem(6, Bt=1, H=2, P=3, N=2, GB=1, GC=2, W=3, T=5)
    flags = 0
    j, k = 2, 3
    y, s_out, c_out = run_verify(q, np.array([j], dtype=np.int32), k, flags)
    T, H, P, N = 5, 2, 3, 2
    xc = full_conv_channels(q, 0, flags).reshape(T, H, P)
    dt, A, Bm, Cm, D, h0 = q["dt"][0], q["A"], q["B"][0], q["C"][0], q["D"], q["state"][0]
    for h in range(H):
        for t in range(T):
            for p in range(P):
                tot = D[h] * xc[t, h, p]
                decay0 = np.exp(A[h] * sum(dt[r, h] for r in range(t + 1)))
                tot += decay0 * sum(Cm[t, h, n] * h0[h, p, n] for n in range(N))
                for s_ in range(t + 1):
                    dec = np.exp(A[h] * sum(dt[r, h] for r in range(s_ + 1, t + 1)))
                    cb = sum(Cm[t, h, n] * Bm[s_, 0, n] for n in range(N))
                    tot += dec * dt[s_, h] * cb * xc[s_, h, p]
                assert y[0, t, h, p] == pytest.approx(tot, rel=1e-12, abs=1e-13)
        for p in range(P):
            for n in range(N):
                tot = np.exp(A[h] * sum(dt[r, h] for r in range(j))) * h0[h, p, n]
                for s_ in range(j):
                    dec = np.exp(A[h] * sum(dt[r, h] for r in range(s_ + 1, j)))
                    tot += dec * dt[s_, h] * xc[s_, h, p] * Bm[s_, 0, n]
                assert s_out[0, h, p, n] == pytest.approx(tot, rel=1e-12, abs=1e-14)
    # conv window after j tokens: the last W-1 = 2 inputs
    np.testing.assert_array_equal(c_out[0], q["x"][0, j - 2:j].reshape(2, H * P))


# --------------------------------------------------------------------------- conv, activation, gate
def test_rolling_conv_equals_full_correlation_and_delta_kernel_is_identity():
    q = small_problem(7, Bt=2, H=1, P=4, N=1, GB=1, GC=1, W=4, T=8)
    Bt, T, H, P = q["x"].shape
    # N=1, h0=0, B=0, C=0, D=1  =>  y_t = xc_t, which isolates the convolution
    over = dict(state=np.zeros_like(q["state"]), B=np.zeros_like(q["B"]), C=np.zeros_like(q["C"]), D=np.ones(H))
    n_prev = np.array([5, 2], dtype=np.int32)
    for flags in (0, CSILU):
        y, _, c_out = run_verify(q, n_prev, 3, flags, **over)
        for b in range(Bt):
            Tb = n_prev[b] + 3
            np.testing.assert_allclose(y[b, :Tb, 0], full_conv_channels(q, b, flags)[:Tb], rtol=1e-13, atol=1e-15)
            hist = np.concatenate([q["conv"][b], q["x"][b, :n_prev[b]].reshape(-1, P)])
            np.testing.assert_array_equal(c_out[b], hist[-3:])
    delta = np.zeros_like(q["cw"])
    delta[:, -1] = 1.0
    y, _, _ = run_verify(q, n_prev, 3, 0, cw=delta, cb=np.zeros_like(q["cb"]), **over)
    np.testing.assert_array_equal(y[0, :8, 0], q["x"][0, :8, 0])
    # a kernel that is 1 on the OLDEST tap returns the input delayed by W-1 = 3 tokens
    oldest = np.zeros_like(q["cw"])
    oldest[:, 0] = 1.0
    y, _, _ = run_verify(q, n_prev, 3, 0, cw=oldest, cb=np.zeros_like(q["cb"]), **over)
    np.testing.assert_array_equal(y[0, 3:8, 0], q["x"][0, 0:5, 0])
    np.testing.assert_array_equal(y[0, 0:3, 0], q["conv"][0].reshape(3, P))


def test_gate_multiplies_by_silu_of_z_and_skip_uses_post_conv_x():
    q = small_problem(8)
    n_prev = np.array([1, 2, 3], dtype=np.int32)
    y0, s0, _ = run_verify(q, n_prev, 4, CSILU)
    y1, s1, _ = run_verify(q, n_prev, 4, CSILU | GATE)
    np.testing.assert_array_equal(s0, s1)
    z = q["z"]
    valid = ~np.isnan(y0)
    np.testing.assert_allclose(y1[valid], (y0 * z / (1 + np.exp(-z)))[valid], rtol=1e-13)
    # D enters as D_h * xc: the difference between two D vectors is (D2-D1) * xc
    D2 = q["D"] + np.array([1.0, -2.0, 0.5, 3.0])
    y2, _, _ = run_verify(q, n_prev, 4, CSILU, D=D2)
    Bt, T, H, P = q["x"].shape
    for b in range(Bt):
        xc = full_conv_channels(q, b, CSILU).reshape(T, H, P)
        Tb = n_prev[b] + 4
        np.testing.assert_allclose((y2 - y0)[b, :Tb], (D2 - q["D"])[None, :, None] * xc[:Tb], rtol=1e-10, atol=1e-12)


def test_group_mapping_head_h_uses_group_h_over_heads_per_group():
    q = small_problem(9, H=4, GB=2, GC=4)
    n_prev = np.array([2, 2, 2], dtype=np.int32)
    y, s_out, _ = run_verify(q, n_prev, 2, 0)
    # changing group 1 of B must change heads 2,3 only
    B2 = q["B"].copy()
    B2[:, :, 1] += 1.0
    y2, s2, _ = run_verify(q, n_prev, 2, 0, B=B2)
    assert np.array_equal(s_out[:, :2], s2[:, :2]) and not np.allclose(s_out[:, 2:], s2[:, 2:])
    # changing group 3 of C must change head 3's outputs only
    C2 = q["C"].copy()
    C2[:, :, 3] += 1.0
    y3, _, _ = run_verify(q, n_prev, 2, 0, C=C2)
    assert np.array_equal(y[:, :4, :3], y3[:, :4, :3]) and not np.allclose(y[:, :4, 3], y3[:, :4, 3])


# --------------------------------------------------------------------------- edges
def test_edges_nothing_accepted_and_pure_advance():
    q = small_problem(10)
    # j = 0 everywhere: cache untouched, outputs still produced for the k drafts
    y, s_out, c_out = run_verify(q, np.zeros(3, dtype=np.int32), 3, GATE | CSILU)
    np.testing.assert_array_equal(s_out, q["state"])
    np.testing.assert_array_equal(c_out, q["conv"])
    assert not np.isnan(y[:, :3]).any() and np.isnan(y[:, 3:]).all()
    # k = 0: pure advance over j tokens equals the sequential run
    n_prev = np.array([5, 0, 7], dtype=np.int32)
    y, s_out, c_out = run_verify(q, n_prev, 0, GATE | CSILU)
    _, s_seq, c_seq = oracle.sequential(q["state"], q["conv"], q["x"], q["dt"], q["B"], q["C"], q["A"], q["D"],
                                        q["cw"], q["cb"], q["z"], n_prev, GATE | CSILU)
    np.testing.assert_allclose(s_out, s_seq, rtol=1e-12, atol=1e-14)
    np.testing.assert_array_equal(c_out, c_seq)
    # j + k beyond the rows that exist is refused
    with pytest.raises(ValueError):
        run_verify(q, np.array([5, 0, 7], dtype=np.int32), 1, 0)


def test_padding_rows_are_never_read():
    s = synth.Shape("pin_pad", Bt=2, H=2, P=4, N=4, GB=1, GC=2, W=4, k=2, act="fp32")
    A, D, cw, cb = synth.layer_params(s)
    st, cv = synth.initial_cache(s)
    r = synth.Rounds(s, synth.token_stream(s, 0, 16))
    r.accept(np.array([1, 2]))
    b = r.batch()
    assert np.isnan(b["x"][0, 3:]).all() and not np.isnan(b["x"][1]).any()
    y, s_out, _ = oracle.verify(st, cv, b["x"], b["dt"], b["B"], b["C"], A, D, cw, cb, b["z"], b["n_prev"], s.k,
                                s.flags)
    assert not np.isnan(s_out).any() and not np.isnan(y[0, :3]).any() and np.isnan(y[0, 3:]).all()


# --------------------------------------------------------------------------- Mamba-1 parameterisation (Algorithm 1)
def m1_problem(seed, **kw):
    """small_problem with a sampling interval per channel, A per (channel, column) and D per channel."""
    q = small_problem(seed, **kw)
    g = np.random.default_rng(seed + 1000)
    Bt, T, H, P = q["x"].shape
    N = q["state"].shape[-1]
    q["dt"] = np.log1p(np.exp(g.standard_normal((Bt, T, H * P)) - 1.0))
    q["A"] = -np.exp(g.uniform(0, np.log(16), (H * P, N)))
    q["D"] = g.standard_normal(H * P)
    return q


def run_verify_m1(q, n_prev, k, flags, **over):
    a = dict(q, **over)
    return oracle.verify_m1(a["state"], a["conv"], a["x"], a["dt"], a["B"], a["C"], a["A"], a["D"],
                            a["cw"], a["cb"], a["z"], n_prev, k, flags)


@pytest.mark.parametrize("flags", [0, GATE | CSILU])
def test_m1_reduces_to_the_per_head_form_when_dt_and_A_are_constant_over_a_head(flags):
    """Algorithm 1 with one interval and one A per head is the form the rest of this file pins."""
    q = small_problem(21)
    Bt, T, H, P = q["x"].shape
    N = q["state"].shape[-1]
    n_prev = np.array([0, 2, 3], dtype=np.int32)
    y0, s0, c0 = run_verify(q, n_prev, 4, flags)
    y1, s1, c1 = run_verify_m1(q, n_prev, 4, flags, dt=np.repeat(q["dt"], P, axis=2),
                               A=np.repeat(q["A"], P)[:, None] * np.ones((1, N)), D=np.repeat(q["D"], P))
    valid = ~np.isnan(y0)
    assert (np.isnan(y1) == np.isnan(y0)).all()
    np.testing.assert_allclose(y1[valid], y0[valid], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(s1, s0, rtol=1e-12, atol=1e-13)
    np.testing.assert_array_equal(c1, c0)


@pytest.mark.parametrize("flags", [0, GATE, CSILU, GATE | CSILU])
def test_m1_multistep_equals_repeated_single_steps(flags):
    q = m1_problem(22)
    Bt, T, H, P = q["x"].shape
    n_prev = np.zeros(Bt, dtype=np.int32)
    y, _, _ = run_verify_m1(q, n_prev, T, flags)
    st, cv = q["state"].copy(), q["conv"].copy()
    for t in range(T):
        y1, st, cv = oracle.step_m1(st, cv, q["x"][:, t], q["dt"][:, t], q["B"][:, t], q["C"][:, t], q["A"], q["D"],
                                    q["cw"], q["cb"], q["z"][:, t], flags)
        np.testing.assert_allclose(y[:, t], y1, rtol=1e-11, atol=1e-12)
    # the snapshot after all tokens is what the single steps arrive at
    _, s_all, c_all = run_verify_m1(q, np.full(Bt, T, dtype=np.int32), 0, flags)
    np.testing.assert_allclose(s_all, st, rtol=1e-11, atol=1e-12)
    np.testing.assert_array_equal(c_all, cv)


def test_m1_unrolled_sums_by_brute_force():
    """y_t[p] = sum_n C_t[n] ( exp(A[c,n] S_{0,t}) h0[p,n] + sum_{s<=t} exp(A[c,n] S_{s,t}) dt_s[c] xc_s[p] B_s[n] ) + D[c] xc_t[p],
    S_{s,t} = sum_{s<r<=t} dt_r[c], written as explicit sums with no recurrence."""
    q = m1_problem(23, Bt=2, H=2, P=3, N=4, GB=1, GC=2, T=5)
    Bt, T, H, P = q["x"].shape
    N = q["state"].shape[-1]
    y, s_out, _ = run_verify_m1(q, np.array([2, 5], dtype=np.int32), 0, 0)
    ylong, _, _ = run_verify_m1(q, np.zeros(Bt, dtype=np.int32), T, 0)
    for b in range(Bt):
        xc = full_conv_channels(q, b, 0)
        for c in range(H * P):
            h, p = divmod(c, P)
            gB, gC = h // (H // 1), h // (H // 2)
            for t in range(T):
                tot = q["D"][c] * xc[t, c]
                for n in range(N):
                    acc = np.exp(q["A"][c, n] * q["dt"][b, :t + 1, c].sum()) * q["state"][b, h, p, n]
                    for s in range(t + 1):
                        acc += np.exp(q["A"][c, n] * q["dt"][b, s + 1:t + 1, c].sum()) * q["dt"][b, s, c] * xc[s, c] * q["B"][b, s, gB, n]
                    tot += q["C"][b, t, gC, n] * acc
                    if t + 1 == (2, 5)[b]:
                        np.testing.assert_allclose(s_out[b, h, p, n], acc, rtol=1e-11, atol=1e-13)
                np.testing.assert_allclose(ylong[b, t, h, p], tot, rtol=1e-11, atol=1e-13)


def test_m1_closed_forms():
    q = m1_problem(24)
    Bt, T, H, P = q["x"].shape
    N = q["state"].shape[-1]
    full = np.full(Bt, T, dtype=np.int32)
    # dt = 0: nothing moves, y = C . h0 + D xc
    y, s, _ = run_verify_m1(q, full, 0, 0, dt=np.zeros_like(q["dt"]))
    np.testing.assert_array_equal(s, q["state"])
    for b in range(Bt):
        xc = full_conv_channels(q, b, 0).reshape(T, H, P)
        for h in range(H):
            want = np.einsum("tn,pn->tp", q["C"][b, :, h // (H // 4)], q["state"][b, h]) + q["D"].reshape(H, P)[h] * xc[:, h]
            np.testing.assert_allclose(y[b, :, h], want, rtol=1e-12, atol=1e-13)
    # B = 0, constant interval per channel: every element decays by exp(A[c,n] T dt[c])
    dtc = np.broadcast_to(q["dt"][:, :1], q["dt"].shape).copy()
    _, s, _ = run_verify_m1(q, full, 0, 0, dt=dtc, B=np.zeros_like(q["B"]))
    want = q["state"] * np.exp(q["A"].reshape(1, H, P, N) * (T * dtc[:, 0].reshape(Bt, H, P, 1)))
    np.testing.assert_allclose(s, want, rtol=1e-12, atol=1e-14)
    # A -> 0: a cumulative sum of rank-one terms dt_t[c] xc_t[p] B_t[n]
    _, s, _ = run_verify_m1(q, full, 0, 0, A=np.zeros_like(q["A"]))
    for b in range(Bt):
        xc = full_conv_channels(q, b, 0).reshape(T, H, P)
        for h in range(H):
            upd = np.einsum("tp,tn->pn", q["dt"][b].reshape(T, H, P)[:, h] * xc[:, h], q["B"][b, :, h // (H // 2)])
            np.testing.assert_allclose(s[b, h], q["state"][b, h] + upd, rtol=1e-12, atol=1e-13)


def test_m1_snapshot_positions_and_untouched_rows():
    q = m1_problem(25)
    Bt, T, H, P = q["x"].shape
    n_prev = np.array([0, 1, 3], dtype=np.int32)
    y, s, c = run_verify_m1(q, n_prev, 3, GATE | CSILU)
    for b in range(Bt):
        assert np.isnan(y[b, n_prev[b] + 3:]).all() and not np.isnan(y[b, :n_prev[b] + 3]).any()
        _, sb, cb = run_verify_m1(q, np.full(Bt, n_prev[b], dtype=np.int32), 0, GATE | CSILU)
        np.testing.assert_allclose(s[b], sb[b], rtol=1e-12, atol=1e-14)
        np.testing.assert_array_equal(c[b], cb[b])
    np.testing.assert_array_equal(s[0], q["state"][0])


# --------------------------------------------------------------------------- softplus of the raw interval
def test_softplus_dt_against_its_identities():
    g = np.random.default_rng(31)
    v = g.uniform(-20, 20, (4, 5, 6))
    bias = g.standard_normal(6)
    sp = oracle.softplus_dt(v, bias)
    u = v + bias
    np.testing.assert_allclose(sp - oracle.softplus_dt(-v, -bias), u, rtol=1e-12, atol=1e-12)      # sp(u) - sp(-u) = u
    np.testing.assert_allclose(np.expm1(sp), np.exp(u), rtol=1e-10)                                 # exp(sp(u)) = 1 + exp(u)
    np.testing.assert_allclose(oracle.softplus_dt(np.zeros(3), np.zeros(3)), np.log(2.0))
    eps = 1e-6                                                                                      # d sp / du = sigmoid
    np.testing.assert_allclose((oracle.softplus_dt(v + eps, bias) - oracle.softplus_dt(v - eps, bias)) / (2 * eps),
                               1.0 / (1.0 + np.exp(-u)), rtol=1e-6, atol=1e-9)
    assert oracle.softplus_dt(np.array([100.0]), np.array([0.0]))[0] == 100.0


# --------------------------------------------------------------------------- gated RMSNorm epilogue
def test_gated_rmsnorm_against_its_definition_and_invariants():
    rng = np.random.default_rng(7)
    H, P = 3, 5
    y = rng.standard_normal((2, 4, H, P))
    w = 1.0 + 0.1 * rng.standard_normal(H * P)
    eps = 1e-5
    out = oracle.gated_rmsnorm(y, w, eps)
    # the definition, element by element in plain Python
    for b in range(2):
        for t in range(4):
            flat = [float(y[b, t, h, p]) for h in range(H) for p in range(P)]
            ms = sum(v * v for v in flat) / len(flat)
            for c, v in enumerate(flat):
                assert abs(out[b, t, c // P, c % P] - w[c] * v / (ms + eps) ** 0.5) < 1e-13
    # unit weight, no eps: every row has mean square exactly one
    unit = oracle.gated_rmsnorm(y, np.ones(H * P), 0.0)
    np.testing.assert_allclose((unit.reshape(8, -1) ** 2).mean(axis=1), 1.0, rtol=1e-13)
    # scale invariance without eps, and the sign of the input survives
    np.testing.assert_allclose(oracle.gated_rmsnorm(37.0 * y, w, 0.0), oracle.gated_rmsnorm(y, w, 0.0), rtol=1e-12)
    np.testing.assert_allclose(oracle.gated_rmsnorm(-y, w, eps), -out, rtol=1e-13)
    # a huge eps turns it into a plain scaling by weight / sqrt(eps)
    big = oracle.gated_rmsnorm(y, w, 1e12)
    np.testing.assert_allclose(big, (w.reshape(H, P) * y) / 1e6, rtol=1e-9)
    # a permutation of the channels permutes the result (the mean runs over all H*P channels, not per head)
    perm = rng.permutation(H * P)
    yp = y.reshape(2, 4, -1)[:, :, perm].reshape(2, 4, H, P)
    np.testing.assert_allclose(oracle.gated_rmsnorm(yp, w[perm], eps).reshape(2, 4, -1), out.reshape(2, 4, -1)[:, :, perm], rtol=1e-13)
    # one row does not touch another; padding rows stay NaN
    y2 = y.copy()
    y2[1, 3] = np.nan
    out2 = oracle.gated_rmsnorm(y2, w, eps)
    assert np.isnan(out2[1, 3]).all()
    np.testing.assert_array_equal(out2[0], out[0])
    np.testing.assert_array_equal(out2[1, :3], out[1, :3])
    with pytest.raises(ValueError):
        oracle.gated_rmsnorm(y, w[:-1], eps)


# --------------------------------------------------------------------------- conv over the B and C channels
def bc_problem(seed, **kw):
    q = small_problem(seed, **kw)
    g = np.random.default_rng(seed + 1000)
    Bt, T, GB, N = q["B"].shape
    GC, W = q["C"].shape[2], q["cw"].shape[1]
    ch = (GB + GC) * N
    q.update(conv_bc=0.5 * g.standard_normal((Bt, W - 1, ch)), cw_bc=g.standard_normal((ch, W)) / 2, cb_bc=0.1 * g.standard_normal(ch))
    return q


def run_verify_bc(q, n_prev, k, flags, **over):
    a = dict(q, **over)
    return oracle.verify_conv_bc(a["state"], a["conv"], a["conv_bc"], a["x"], a["dt"], a["B"], a["C"], a["A"], a["D"], a["cw"], a["cb"],
                                 a["cw_bc"], a["cb_bc"], a["z"], n_prev, k, flags)


def test_conv_rows_against_numpy_correlate_and_its_special_kernels():
    g = np.random.default_rng(5)
    Bt, T, Ch, W = 2, 9, 6, 4
    rows, window = g.standard_normal((Bt, T, Ch)), g.standard_normal((Bt, W - 1, Ch))
    taps, bias = g.standard_normal((Ch, W)), g.standard_normal(Ch)
    n_prev = np.array([4, 0], dtype=np.int32)
    out, win = oracle.conv_rows(rows, window, taps, bias, n_prev, 5, False)
    for b in range(Bt):
        Tb = n_prev[b] + 5
        for c in range(Ch):
            hist = np.concatenate([window[b, :, c], rows[b, :, c]])
            full = np.correlate(hist, taps[c], mode="valid") + bias[c]     # tap W-1 on the current token
            np.testing.assert_allclose(out[b, :Tb, c], full[:Tb], rtol=1e-13, atol=1e-14)
        assert np.isnan(out[b, Tb:]).all()
        hist = np.concatenate([window[b], rows[b, :n_prev[b]]])
        np.testing.assert_array_equal(win[b], hist[-(W - 1):])              # window at the verified position
    silu, _ = oracle.conv_rows(rows, window, taps, bias, n_prev, 5, True)
    np.testing.assert_allclose(silu[0, :9], out[0, :9] / (1 + np.exp(-out[0, :9])), rtol=1e-13)
    delta = np.zeros((Ch, W))
    delta[:, -1] = 1.0
    ident, _ = oracle.conv_rows(rows, window, delta, np.zeros(Ch), n_prev, 5, False)
    np.testing.assert_array_equal(ident[0, :9], rows[0, :9])
    oldest = np.zeros((Ch, W))
    oldest[:, 0] = 1.0
    delayed, _ = oracle.conv_rows(rows, window, oldest, np.zeros(Ch), n_prev, 5, False)
    np.testing.assert_array_equal(delayed[0, 3:9], rows[0, 0:6])
    np.testing.assert_array_equal(delayed[0, 0:3], window[0])


def test_conv_over_b_and_c_reduces_to_the_plain_call_and_chains_like_it():
    q = bc_problem(31)
    n_prev = np.array([0, 2, 3], dtype=np.int32)
    # identity taps and no activation: B and C pass through unchanged, the call is the pinned one
    ch, W = q["cw_bc"].shape
    delta = np.zeros((ch, W))
    delta[:, -1] = 1.0
    y0, s0, c0 = run_verify(q, n_prev, 3, GATE)
    y1, s1, c1, w1 = run_verify_bc(q, n_prev, 3, GATE, cw_bc=delta, cb_bc=np.zeros(ch))
    np.testing.assert_array_equal(np.nan_to_num(y1), np.nan_to_num(y0))
    np.testing.assert_array_equal(s1, s0)
    np.testing.assert_array_equal(c1, c0)
    # with real taps: the recurrence sees exactly conv_rows' outputs (B channels first, then C)
    Bt, T, GB, N = q["B"].shape
    GC = q["C"].shape[2]
    rows = np.concatenate([q["B"].reshape(Bt, T, -1), q["C"].reshape(Bt, T, -1)], axis=2)
    out, win = oracle.conv_rows(rows, q["conv_bc"], q["cw_bc"], q["cb_bc"], n_prev, 3, True)
    out = np.nan_to_num(out)
    y2, s2, c2, w2 = run_verify_bc(q, n_prev, 3, GATE | CSILU)
    y3, s3, c3 = run_verify(q, n_prev, 3, GATE | CSILU, B=out[:, :, :GB * N].reshape(Bt, T, GB, N), C=out[:, :, GB * N:].reshape(Bt, T, GC, N))
    np.testing.assert_array_equal(np.nan_to_num(y2), np.nan_to_num(y3))
    np.testing.assert_array_equal(s2, s3)
    np.testing.assert_array_equal(w2, win)
    # a call that replays j tokens and drafts k equals a call over the j tokens followed by one over the k drafts
    # from the caches the first one left (state, both conv windows)
    ya, sa, ca, wa = run_verify_bc(q, n_prev, 3, GATE | CSILU)
    zero = np.zeros(3, dtype=np.int32)
    for b in range(3):
        j = int(n_prev[b])
        sl = slice(b, b + 1)
        qa = {k_: (v[sl] if k_ in ("state", "conv", "conv_bc", "x", "z", "dt", "B", "C") else v) for k_, v in q.items()}
        nb = np.array([j], dtype=np.int32)
        _, s_first, c_first, w_first = run_verify_bc(qa, nb, 0, GATE | CSILU)
        np.testing.assert_allclose(s_first, sa[sl], rtol=1e-13, atol=1e-15)
        np.testing.assert_array_equal(w_first, wa[sl])
        qb = dict(qa, state=s_first, conv=c_first, conv_bc=w_first)
        for name in ("x", "z", "dt", "B", "C"):
            qb[name] = np.concatenate([qa[name][:, j:], np.zeros_like(qa[name][:, :j])], axis=1)
        y_second, _, _, _ = run_verify_bc(qb, np.zeros(1, dtype=np.int32), 3, GATE | CSILU)
        np.testing.assert_allclose(y_second[0, :3], ya[b, j:j + 3], rtol=1e-12, atol=1e-13)
