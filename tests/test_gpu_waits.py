"""The streaming kernel's give-up path, run for real but safely: a test-only build of the library (same sources,
two macros) whose waits give up after about a millisecond and in which the barrier of the small inputs expects
16 transaction bytes more than are ever requested.  Every copy the kernel starts still lands; the barrier
just never completes, the consumers' bounded wait runs out, the kernel sets MAMBA_SPEC_STATUS_COPY_TIMEOUT,
lets what is in flight land and returns.  Nothing traps and the context stays usable."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2408_15237_b200 import synth

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_and_the_kernel_returns():
    from paper_2408_15237_b200 import binding, build
    import harness as h
    lib = ctypes.CDLL(str(build.build_wait_test_library()))
    vp, i32 = ctypes.c_void_p, ctypes.c_int32
    lib.mamba_spec_init.argtypes = [ctypes.POINTER(binding.Config), ctypes.POINTER(vp)]
    lib.mamba_spec_verify.argtypes = [vp] * 10 + [i32, ctypes.POINTER(binding.IO)]
    lib.mamba_spec_status.argtypes = [vp, ctypes.POINTER(i32)]
    lib.mamba_spec_last_kernel.restype = ctypes.c_char_p
    lib.mamba_spec_last_kernel.argtypes = [vp]
    lib.mamba_spec_destroy.argtypes = [vp]
    s = synth.SWEEP[(4, 4)]
    cfg = binding.Config(s.Bt, 1, s.H, s.P, s.N, s.GB, s.GC, s.W, s.k, binding.DTYPE_BF16, s.flags, 0, binding.KERNEL_STREAM)
    ctx = vp()
    assert lib.mamba_spec_init(ctypes.byref(cfg), ctypes.byref(ctx)) == 0
    lay = h.Layer(s)
    r = synth.Rounds(s, synth.token_stream(s, 0, 3 * s.k), first_j=2)
    b = r.batch()
    ad = torch.bfloat16
    t = {n: h.dev(np.nan_to_num(b[n]), ad) for n in ("x", "z", "dt", "B", "C")}
    y = torch.full(t["x"].shape, float("nan"), device="cuda", dtype=ad)
    n_prev = h.dev(b["n_prev"], torch.int32)
    state0, conv0 = lay.state.clone(), lay.conv.clone()
    io = binding.IO(lay.cw.data_ptr(), lay.cb.data_ptr(), t["z"].data_ptr(), y.data_ptr(), s.Bt, 0, s.t_max,
                    torch.cuda.current_stream().cuda_stream, None, None, None)
    rc = lib.mamba_spec_verify(ctx, lay.state.data_ptr(), lay.conv.data_ptr(), t["x"].data_ptr(), t["dt"].data_ptr(),
                               t["B"].data_ptr(), t["C"].data_ptr(), lay.A.data_ptr(), lay.D.data_ptr(), n_prev.data_ptr(), s.k,
                               ctypes.byref(io))
    assert rc == 0 and lib.mamba_spec_last_kernel(ctx).decode().startswith("stream<")
    flags = i32(-1)
    assert lib.mamba_spec_status(ctx, ctypes.byref(flags)) == 0          # synchronises: the kernel has returned
    assert flags.value & binding.STATUS_COPY_TIMEOUT
    torch.cuda.synchronize()                                              # no fault: the device still answers
    # the wait that ran out sits in front of everything: nothing was computed, nothing was written
    assert torch.isnan(y.float()).all()
    assert torch.equal(lay.state, state0) and torch.equal(lay.conv, conv0)
    # the status word was cleared by the read, and the context still takes calls
    assert lib.mamba_spec_status(ctx, ctypes.byref(flags)) == 0 and flags.value == 0
    lib.mamba_spec_destroy(ctx)
    # and the product library, in the same process, computes as ever on the same device
    ver = h.make_verifier(s, 2)
    y_gpu = lay.gpu_verify(ver, b, s.k)
    y_ref = lay.oracle_verify(b, s.k)
    lay.check(y_gpu, y_ref, h.TOL[s.act], "after the timed-out launch")
    assert ver.status() == 0
    ver.close()
