#!/usr/bin/env python
"""Benchmark of the multi-step Mamba verification step (speculative decoding, Sec. 4.2-4.3).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--sweep]

Workload of the default run: the hybrid-stack decode loop -- 24 Mamba layers of the
Llama3-8B-derived shape (H=32, P=128, N=128, B from 8 groups, C per head, conv width 4), batch 16,
k=4 draft tokens, per-sequence acceptance lengths geometric(p=0.4) capped at k.  One *step* is one
speculation round: 24 verify launches (one per layer, pending lengths taken from the last commit)
plus the commit.  Eight distinct rounds of inputs are resident in HBM and captured as CUDA graphs;
step i replays round i mod 8.  A step reads 768 MiB of fp32 state, six times the L2, so every
launch streams its state from HBM.

Prints one JSON line (see the keys below).  `--impl reference` times the fp64 CPU oracle instead
(a deliberately plain program; the ratio to it says nothing about kernel quality).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2408_15237_b200 import synth  # noqa: E402

METRIC = "verified_draft_tokens_per_s_per_mamba_layer"
UNIT = "tokens/s/layer"
N_ROUND_SETS = 8
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "verify_stream_dram_traffic.txt")
KERNEL_SOURCES = ("paper_2408_15237_b200/csrc/verify_stream.cu", "paper_2408_15237_b200/csrc/common.cuh")


def kernel_source_hash():
    import hashlib
    hsh = hashlib.sha256()
    for rel in KERNEL_SOURCES:
        with open(os.path.join(ROOT, rel), "rb") as f:
            hsh.update(f.read())
    return hsh.hexdigest()[:16]


def measured_traffic(plan_name):
    """DRAM bytes per launch of the streaming kernel from the kept ncu summary, or None when that summary was taken
    with another plan or another version of the kernel's source (then it says nothing about this run)."""
    rec = {}
    try:
        with open(TRAFFIC_FILE) as f:
            for line in f:
                if "=" in line and not line.lstrip().startswith("#"):
                    k, v = line.split("=", 1)
                    rec[k.strip()] = v.strip()
    except OSError:
        return None, None
    if rec.get("source_sha256_16") != kernel_source_hash() or rec.get("plan") != plan_name:
        return None, None
    try:
        rd, wr = float(rec["dram_bytes_read_per_launch"]), float(rec["dram_bytes_write_per_launch"])
    except (KeyError, ValueError):
        return None, None
    return rd + wr, {"dram_bytes_read": rd, "dram_bytes_write": wr, "capture": rec.get("capture", "")}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, plain copy)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


def algorithmic_bytes(s, n_prev, k):
    """Bytes one verify launch must move: state read (+ write where tokens were accepted), the token
    rows of x, z, y, B, C, dt, and the conv window read (+ written).  Parameters are not counted."""
    act = 2 if s.act == "bf16" else 4
    n_prev = np.asarray(n_prev, dtype=np.int64)
    T = n_prev + k
    wrote = (n_prev > 0).astype(np.int64)
    per_head = (4 * s.P * s.N * (1 + wrote) + T * 3 * act * s.P + T * act * s.N * (s.GB + s.GC) / s.H + T * act
                + (1 + wrote) * act * s.P * (s.W - 1))
    return float(per_head.sum() * s.H)


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.samples, self.reasons, self.max_mhz, self.ok = [], set(), None, False
        self._stop_evt = threading.Event()
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20,
                 "hw_power_brake": 0x80}
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for n, bit in names.items():
                    if r & bit:
                        self.reasons.add(n)
            except Exception:
                pass
            time.sleep(0.01)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


class Stack:
    """Device-resident decode-loop workload: per-layer caches and parameters, N_ROUND_SETS rounds of token slabs."""

    def __init__(self, s, device):
        from paper_2408_15237_b200 import binding
        self.s, self.binding = s, binding
        # pending lengths come from commit(), except where another model accepted the tokens (k_prev set)
        self.explicit_n_prev = s.k_prev > 0
        self.ver = binding.Verifier(s.Bt, s.H, s.P, s.N, s.GB, s.GC, s.W, max(s.k, s.k_prev), act=s.act, flags=s.flags,
                                    n_layers=s.n_layers, device=device)
        g = torch.Generator(device="cuda")
        g.manual_seed(synth.BASE_SEED)
        bf = torch.bfloat16
        rn = lambda *shape, std=1.0: torch.randn(*shape, generator=g, device="cuda", dtype=torch.float32) * std
        self.layers = []
        for _ in range(s.n_layers):
            lay = dict(
                state=rn(s.Bt, s.H, s.P, s.N, std=0.1), conv=rn(s.Bt, s.W - 1, s.H * s.P, std=0.1).to(bf),
                A=-torch.exp(torch.rand(s.H, generator=g, device="cuda") * np.log(16.0)), D=rn(s.H),
                cw=rn(s.H * s.P, s.W, std=s.W ** -0.5), cb=rn(s.H * s.P, std=0.1), rounds=[])
            for _r in range(N_ROUND_SETS):
                lay["rounds"].append(dict(
                    x=rn(s.Bt, s.t_max, s.H, s.P).to(bf), z=rn(s.Bt, s.t_max, s.H, s.P).to(bf),
                    dt=torch.nn.functional.softplus(rn(s.Bt, s.t_max, s.H) - 2.0).to(bf),
                    B=rn(s.Bt, s.t_max, s.GB, s.N, std=s.N ** -0.5).to(bf),
                    C=rn(s.Bt, s.t_max, s.GC, s.N, std=s.N ** -0.5).to(bf),
                    y=torch.zeros(s.Bt, s.t_max, s.H, s.P, device="cuda", dtype=bf)))
            if s.flags & synth.FLAG_STATE_K:   # second snapshot (the cache after all tokens) wanted as well
                lay["state_k"], lay["conv_k"] = torch.empty_like(lay["state"]), torch.empty_like(lay["conv"])
            self.layers.append(lay)
        # acceptance lengths of round r are the pending lengths of round r+1 (cyclically)
        self.accept_np = [synth.acceptance(s, r) for r in range(N_ROUND_SETS)]
        self.accept = [torch.from_numpy(a).cuda() for a in self.accept_np]
        self.graphs = None

    def n_prev_of_round(self, r):
        return self.accept_np[(r - 1) % N_ROUND_SETS]

    def run_round(self, r):
        s, v = self.s, self.ver
        for l, lay in enumerate(self.layers):
            t = lay["rounds"][r]
            v.verify(lay["state"], lay["conv"], t["x"], t["dt"], t["B"], t["C"], lay["A"], lay["D"], lay["cw"], lay["cb"],
                     t["z"], t["y"], self.accept[(r - 1) % N_ROUND_SETS] if self.explicit_n_prev else None, s.k, layer=l,
                     state_k=lay.get("state_k"), conv_state_k=lay.get("conv_k"))
        if not self.explicit_n_prev:
            v.commit(self.accept[r])

    def capture(self):
        if not self.explicit_n_prev:
            self.ver.commit(self.accept[N_ROUND_SETS - 1])
        for r in range(N_ROUND_SETS):       # plain runs first: function attributes get set outside capture
            self.run_round(r)
        torch.cuda.synchronize()
        self.graphs = []
        for r in range(N_ROUND_SETS):
            gph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gph):
                self.run_round(r)
            self.graphs.append(gph)
        torch.cuda.synchronize()

    def step(self, i):
        self.graphs[i % N_ROUND_SETS].replay()


class HostStack:
    """End-to-end leg: the per-step tensors live in pinned host memory and cross PCIe inside the timed region.

    The layers of a step are independent calls of mamba_spec_verify_host.  They are spread over N_HOST_STREAMS
    streams, each with its own library context (a context owns one set of device staging buffers), so that
    one layer's host-to-device copies overlap another layer's kernel and device-to-host copy.  The side
    streams start after, and the timed stream ends after, everything of the step (event dependencies), so
    the CUDA events around the steps on the current stream bracket all of it.
    """

    N_HOST_STREAMS = 4

    def __init__(self, stack, n_streams=0):
        self.st = stack
        s, b = stack.s, stack.binding
        self.host = []
        for lay in stack.layers:
            rounds = []
            for t in lay["rounds"][:2]:
                h = {n: t[n].cpu().pin_memory() for n in ("x", "z", "dt", "B", "C")}
                h["y"] = torch.empty(t["y"].shape, dtype=t["y"].dtype).pin_memory()
                rounds.append(h)
            self.host.append(rounds)
        self.n_prev = [torch.from_numpy(stack.n_prev_of_round(r).copy()).pin_memory() for r in range(2)]
        one = self.host[0][0]
        self.h2d = sum(one[n].numel() * one[n].element_size() for n in ("x", "z", "dt", "B", "C")) * s.n_layers \
            + 4 * s.Bt * s.n_layers
        self.d2h = one["y"].numel() * one["y"].element_size() * s.n_layers
        self.streams = [torch.cuda.Stream() for _ in range(n_streams if n_streams > 0 else self.N_HOST_STREAMS)]
        self.vers = [b.Verifier(s.Bt, s.H, s.P, s.N, s.GB, s.GC, s.W, s.k, act=s.act, flags=s.flags, n_layers=s.n_layers,
                                device=torch.cuda.current_device()) for _ in self.streams]

    def step(self, i):
        st, b = self.st, self.st.binding
        s, r = st.s, i % 2
        main = torch.cuda.current_stream()
        for side in self.streams:
            side.wait_stream(main)
        for l, lay in enumerate(st.layers):
            h = self.host[l][r]
            q = l % len(self.streams)
            io = b.IO(lay["cw"].data_ptr(), lay["cb"].data_ptr(), h["z"].data_ptr(), h["y"].data_ptr(), s.Bt, l, s.t_max,
                      self.streams[q].cuda_stream)
            b.mamba_spec_verify_host(self.vers[q].ctx, lay["state"], lay["conv"], h["x"], h["dt"], h["B"], h["C"], lay["A"],
                                     lay["D"], self.n_prev[r], s.k, io)
        for side in self.streams:
            main.wait_stream(side)


def max_over_ranks(ms, device):
    """Largest per-rank time of the job (every rank gets it); one rank: the value itself."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([float(ms)], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(world, batch, k, n_layers, ms_per_step):
    """Whole-job throughput: every rank verifies batch*k draft tokens in each of n_layers launches per step."""
    return world * batch * k * n_layers / (ms_per_step * 1e-3)


def timed(fn, steps, warmup, dist_barrier):
    for i in range(warmup):
        fn(i)
    torch.cuda.synchronize()
    dist_barrier()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0.record()
    for i in range(steps):
        fn(warmup + i)
    t1.record()
    torch.cuda.synchronize()
    dist_barrier()
    return t0.elapsed_time(t1)  # ms


def eager_launch_ms(stack, reps=5):
    """Per-launch duration without a graph: the layers' verify calls of a round issued one after the other through
    the binding (tensor maps come from the context's cache), one event pair around each round's launches."""
    s, v = stack.s, stack.ver
    times = []
    for _ in range(reps):
        for r in range(N_ROUND_SETS):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for l, lay in enumerate(stack.layers):
                t = lay["rounds"][r]
                v.verify(lay["state"], lay["conv"], t["x"], t["dt"], t["B"], t["C"], lay["A"], lay["D"], lay["cw"],
                         lay["cb"], t["z"], t["y"], None, s.k, layer=l)
            e1.record()
            times.append((e0, e1))
            v.commit(stack.accept[r])
    torch.cuda.synchronize()
    return float(np.median([a.elapsed_time(b) for a, b in times])) / len(stack.layers)


def cpu_oracle_sample(s, calls, threads, gpu_check=None):
    """Times the fp64 oracle, as it stands, on `calls` verify calls of one layer of the workload.  `gpu_check`, if
    given, gets the inputs and the oracle's results of the untimed first call (a parity spot check of the library
    on the workload's own shape, outside every timed region)."""
    import oracle
    A, D, cw, cb = synth.layer_params(s, 0)
    st, cv = synth.initial_cache(s, 0)
    stream = synth.token_stream(s, 0, 4 * s.t_max)
    r = synth.Rounds(s, stream, wrap=True)
    r.accept(synth.acceptance(s, 0))
    b = r.batch()      # one untimed call: compiles/loads the C library and touches the buffers
    ref = oracle.verify(st, cv, b["x"], b["dt"], b["B"], b["C"], A, D, cw, cb, b["z"], b["n_prev"], s.k, s.flags,
                        threads=threads)
    if gpu_check is not None:
        gpu_check(dict(A=A, D=D, cw=cw, cb=cb, state=st, conv=cv, batch=b), ref)
    per_call = []
    for c in range(calls):
        b = r.batch()
        t0 = time.perf_counter()
        oracle.verify(st, cv, b["x"], b["dt"], b["B"], b["C"], A, D, cw, cb, b["z"], b["n_prev"], s.k, s.flags,
                      threads=threads)
        per_call.append(time.perf_counter() - t0)
        r.accept(synth.acceptance(s, c + 1))
    return per_call


def parity_spot_check(s, out):
    """Returns a callback for cpu_oracle_sample: runs the library on the same inputs and records the relative L2
    errors of y (against the oracle rounded to the output precision and unrounded) and of the committed state."""
    def check(inp, ref):
        from paper_2408_15237_b200 import binding
        y_ref, st_ref, _ = ref
        ad = torch.bfloat16 if s.act == "bf16" else torch.float32
        dev = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a)).to(device="cuda", dtype=dt)
        ver = binding.Verifier(s.Bt, s.H, s.P, s.N, s.GB, s.GC, s.W, s.k, act=s.act, flags=s.flags)
        b = inp["batch"]
        t = {n: dev(np.nan_to_num(b[n]), ad) for n in ("x", "z", "dt", "B", "C")}
        y = torch.zeros(t["x"].shape, device="cuda", dtype=ad)
        state, conv = dev(inp["state"], torch.float32), dev(inp["conv"], ad)
        ver.verify(state, conv, t["x"], t["dt"], t["B"], t["C"], dev(inp["A"], torch.float32), dev(inp["D"], torch.float32),
                   dev(inp["cw"], torch.float32), dev(inp["cb"], torch.float32), t["z"], y, dev(b["n_prev"], torch.int32), s.k)
        torch.cuda.synchronize()
        valid = ~np.isnan(y_ref)
        yg = y.float().cpu().numpy().astype(np.float64)
        rel = lambda a, w: float(np.linalg.norm(a - w) / np.linalg.norm(w))
        yq = synth.round_bf16(np.nan_to_num(y_ref).astype(np.float32)).astype(np.float64) if s.act == "bf16" else y_ref
        out.update({"kernel": ver.last_kernel, "y_rel_l2_vs_unrounded_oracle": rel(yg[valid], y_ref[valid]),
                    "y_rel_l2_vs_oracle_rounded_to_output_dtype": rel(yg[valid], yq[valid]),
                    "state_rel_l2": rel(state.cpu().numpy().astype(np.float64), st_ref), "device_status": ver.status()})
        ver.close()
    return check


def run_reference(args, s, rank):
    import oracle
    if rank != 0:
        return
    threads = oracle.host_threads()
    calls = cpu_oracle_sample(s, args.warmup + args.steps, threads)[args.warmup:]
    sec = float(np.mean(calls))
    value = s.Bt * s.k / sec
    sample = (f"each step = one oracle verify call of one layer (batch {s.Bt}, k={s.k}, T_b=j_b+k rows), "
              f"{threads} OpenMP threads over (sequence, head)")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(s), "note": "fp64 CPU oracle, one layer-call per step"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def workload_name(s):
    return (f"config4 hybrid-stack decode loop: {s.n_layers} Mamba layers, H={s.H} P={s.P} N={s.N} G_B={s.GB} "
            f"G_C={s.GC} W={s.W}, batch {s.Bt}, k={s.k}, acceptance geometric(p={s.accept_p}) capped at k")


def run_sweep(args):
    """Config-2/3 sweep: one layer shape at several batch sizes and draft lengths, 24 rotating buffer sets."""
    from paper_2408_15237_b200 import binding  # noqa: F401
    peak, peak_src = measured_peaks()
    rows = []
    shapes = [synth.SWEEP[key] for key in sorted(synth.SWEEP)] + [synth.CONFIGS[3]]
    for s0 in shapes:
        s = synth.replace(s0, n_layers=24, accept=s0.accept if s0.accept == "geometric" else "uniform")
        st = Stack(s, 0)
        st.capture()
        ms = timed(st.step, args.steps, args.warmup, lambda: None)
        bytes_step = sum(algorithmic_bytes(s, st.n_prev_of_round(r), s.k) for r in range(N_ROUND_SETS)) / N_ROUND_SETS \
            * s.n_layers
        gbs = bytes_step * args.steps / (ms * 1e-3) / 1e9
        rows.append({"shape": s0.name, "batch": s.Bt, "k": s.k, "us_per_launch": ms * 1e3 / args.steps / s.n_layers,
                     "tokens_per_s_per_layer": s.Bt * s.k * s.n_layers * args.steps / (ms * 1e-3),
                     "GBps": gbs, "frac_of_copy_peak": gbs / peak, "frac_of_8TBps": gbs / 8000.0,
                     "kernel": st.ver.last_kernel})
        print(json.dumps(rows[-1]), flush=True)
        st.ver.close()
        del st
        torch.cuda.empty_cache()
    return rows


def run_multistep(args):
    """Second workload (Fig. 3 of the paper): 32 tokens through the multi-step kernel as a function of the step size.

    Every call starts from the cached state (nothing pending, j = 0) and takes `step` new tokens; 32 / step calls
    make 32 tokens.  Reported per (batch, step): microseconds per call and per 32 tokens of one layer.
    """
    from paper_2408_15237_b200 import binding  # noqa: F401
    rows = []
    for bt in (1, 4, 16, 64):
        for step in (1, 2, 4, 8, 16, 32):
            s = synth.replace(synth.llama8b_layer(f"multistep_b{bt}_s{step}", bt, step), n_layers=8, accept="none", t_rows=step)
            st = Stack(s, 0)
            st.capture()
            steps = max(20, args.steps // 10)
            ms = timed(st.step, steps, args.warmup, lambda: None)
            us_call = ms * 1e3 / steps / s.n_layers
            rows.append({"batch": bt, "step": step, "us_per_call": us_call, "us_per_32_tokens": us_call * 32 / step,
                         "kernel": st.ver.last_kernel})
            print(json.dumps(rows[-1]), flush=True)
            st.ver.close()
            del st
            torch.cuda.empty_cache()
    return rows


def run_draft(args):
    """Third workload: the draft model's step (Sec. 4.3): one launch folds the tokens the verifier accepted last
    round (geometric(0.4), at most 4) into the cache and decodes one token.  130M-like layer shape."""
    from paper_2408_15237_b200 import binding  # noqa: F401
    peak, _ = measured_peaks()
    rows = []
    for bt in (1, 4, 16, 64):
        s = synth.Shape(f"draft_b{bt}", Bt=bt, H=24, P=64, N=128, GB=1, GC=1, W=4, k=1, act="bf16", n_layers=24,
                        accept="geometric", accept_p=0.4, t_rows=5, k_prev=4)
        st = Stack(s, 0)
        st.capture()
        ms = timed(st.step, args.steps, args.warmup, lambda: None)
        bytes_step = sum(algorithmic_bytes(s, st.n_prev_of_round(r), s.k) for r in range(N_ROUND_SETS)) / N_ROUND_SETS \
            * s.n_layers
        gbs = bytes_step * args.steps / (ms * 1e-3) / 1e9
        rows.append({"batch": bt, "us_per_launch": ms * 1e3 / args.steps / s.n_layers, "GBps": gbs,
                     "frac_of_copy_peak": gbs / peak, "kernel": st.ver.last_kernel})
        print(json.dumps(rows[-1]), flush=True)
        st.ver.close()
        del st
        torch.cuda.empty_cache()
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sweep", action="store_true", help="batch x k sweep on one GPU instead of the default workload")
    ap.add_argument("--multistep", action="store_true", help="32 tokens vs step size (the paper's Fig. 3 workload) instead")
    ap.add_argument("--draft", action="store_true", help="the draft model's step (replay + one token) instead")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--host-streams", type=int, default=0, help="streams of the end-to-end leg (default %d)" % HostStack.N_HOST_STREAMS)
    ap.add_argument("--profile", action="store_true",
                    help="small case for ncu: --layers layers of the workload shape, eager launches only, no JSON line")
    ap.add_argument("--layers", type=int, default=0, help="with --profile: number of layers (default 4)")
    ap.add_argument("--batch", type=int, default=0, help="with --profile: batch size (default: the workload's)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    s = synth.CONFIGS[4]
    if args.profile:
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device")
        s = synth.replace(s, n_layers=args.layers or 4, Bt=args.batch or s.Bt)
        stack = Stack(s, 0)
        stack.ver.commit(stack.accept[N_ROUND_SETS - 1])
        for i in range(args.warmup + args.steps):
            stack.run_round(i % N_ROUND_SETS)
        torch.cuda.synchronize()
        print(f"profile run: {stack.ver.launches} launches, kernel {stack.ver.last_kernel}, status {stack.ver.status()}")
        return
    if args.gpus > 1 and "RANK" not in os.environ and not (args.sweep or args.multistep or args.draft):
        # started plainly with --gpus N: become N ranks, one per GPU (replicas: the path does not shard)
        import socket
        import subprocess
        with socket.socket() as sock:
            sock.bind(("127.0.0.1", 0))
            port = sock.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1",
               "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        raise SystemExit(subprocess.call(cmd))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, s, rank)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the verification step has no CPU path")
    torch.cuda.set_device(local)
    if args.sweep:
        run_sweep(args)
        return
    if args.multistep:
        run_multistep(args)
        return
    if args.draft:
        run_draft(args)
        return

    use_dist = world > 1
    if use_dist:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        barrier = lambda: dist.barrier()
    else:
        barrier = lambda: None

    stack = Stack(s, local)
    stack.capture()
    sampler = ClockSampler(physical_gpu_index(local))
    sampler.start()
    ms = timed(stack.step, args.steps, args.warmup, barrier)
    clocks = sampler.stop()
    ms = max_over_ranks(ms, "cuda")
    status = stack.ver.status()

    ms_per_step = ms / args.steps
    value = job_value(world, s.Bt, s.k, s.n_layers, ms_per_step)
    peak, peak_src = measured_peaks()
    bytes_launch = float(np.mean([algorithmic_bytes(s, stack.n_prev_of_round(r), s.k) for r in range(N_ROUND_SETS)]))
    us_launch = ms_per_step * 1e3 / s.n_layers
    achieved = bytes_launch / (us_launch * 1e-6) / 1e9
    eager_ms = eager_launch_ms(stack)

    host = HostStack(stack, args.host_streams)
    e2e_steps = max(3, min(args.steps, 30))
    ms_e2e = timed(host.step, e2e_steps, 3, barrier)
    ms_e2e = max_over_ranks(ms_e2e, "cuda")
    e2e_value = job_value(world, s.Bt, s.k, s.n_layers, ms_e2e / e2e_steps)

    cpu, spot = None, {}
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        threads = oracle.host_threads()
        calls = cpu_oracle_sample(s, 12, threads, gpu_check=parity_spot_check(s, spot))
        sec = float(np.mean(calls[2:]))
        cpu = {"value": s.Bt * s.k / sec, "unit": UNIT, "cores": threads, "kind": "oracle",
               "sample": f"10 verify calls of one layer of the workload (batch {s.Bt}, k={s.k}), fp64, "
                         f"{threads} OpenMP threads over (sequence, head); {sec * 1e3:.1f} ms per call"}

    traffic, traffic_detail = measured_traffic(stack.ver.last_kernel)
    if rank == 0:
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": workload_name(s), "step": f"{s.n_layers} verify launches + 1 commit, replayed as a CUDA graph",
                       "l2": f"inputs larger than L2: {s.n_layers * s.Bt * s.H * s.P * s.N * 4 / 2**20:.0f} MiB of state per step",
                       "replicas": "each GPU runs the whole workload (no sharding, no collective)" if world > 1 else "single GPU",
                       "kernel": stack.ver.last_kernel, "device_status": status},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": traffic, "traffic_detail": traffic_detail, "peak_source": peak_src,
                         "algorithmic_bytes_per_launch": bytes_launch,
                         "us_per_launch": us_launch, "us_per_launch_eager": eager_ms * 1e3,
                         "frac_of_8TBps": achieved / 8000.0},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": host.h2d, "d2h_bytes_per_step": host.d2h,
                    "steps": e2e_steps, "ms_per_step": ms_e2e / e2e_steps},
            "gpu_launches": args.steps * (s.n_layers + 1),
            "clocks": clocks,
        }
        if cpu:
            out["cpu_baseline"] = cpu
        if spot:
            out["parity_spot_check"] = spot
        print(json.dumps(out))
    stack.ver.close()
    if use_dist:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
