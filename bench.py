#!/usr/bin/env python
"""Benchmark of the fused packed KD forward+backward step (one JSON line).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config c2|c3|c4|c5]

A step is one pass of the whole hot path over one synthetic batch: LM-head tiles with
online softmax, per-token merge, gradient tiles, dW and dH contractions, then the
segment reductions and the Delta-IFD selection.  The default workload is the ~1B-student
shape the metric is quoted on (c2: T=8192 packed tokens, d=1536, V=151,936, bf16, tau=1);
--config picks one of the other full-size shapes.  `value` is packed tokens/s with the
inputs resident in HBM; `e2e` is the same step through the host-buffer entry point
(host->device copies of hidden states, teacher logits, boundaries, mask and labels and
the device->host read of the per-token losses inside the timed region).

After the timed loop the same loop runs once more with the library's phase events
attached, clocks sampled: `roofline` is the dominant launch group as timed there (so
its time is part of a sustained step, not of a cold single launch), `phase_ms` /
`phase_mcycles` / `tensor_pipe_frac_at_loop_clock` give every group's time, SM cycles
and tensor-pipe utilisation at the clock the loop ran at.

With N > 1 (launched under torch.distributed.run) every rank runs an independent
replica on its own GPU - the path has no collective - and `value` is the sum over
ranks divided by the slowest rank's time.

`--impl reference` times the CPU oracle on the host cores on a bounded sample of the
same workload (the paper ships no implementation to run).
"""

from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np
import torch

# The benchmark configurations.  c2 is the headline (the ~1B-student shape the metric is quoted
# on); c3-c5 are the other full-size shapes, selectable with --config.
WORKLOADS = {
    "c2": dict(name="c2_1b_student", T=8192, d=1536, V=151_936, tau=1.0, make="config2_1b", seed_base=2000),
    "c3": dict(name="c3_packed_rows", T=32768, d=2048, V=151_936, tau=2.0, make="config3_rows", seed_base=3000),
    "c4": dict(name="c4_short_samples", T=16384, d=1536, V=151_936, tau=1.0, make="config4_short", seed_base=4000),
    "c5": dict(name="c5_large_step", T=65536, d=4096, V=151_936, tau=1.0, make="config5_large", seed_base=5000),
}
WORKLOAD = WORKLOADS["c2"]
METRIC = "packed tokens/sec, fused KD fwd+bwd"
UNIT = "tokens/s"


# DRAM bytes (read + write) of one launch of each tensor kernel on the c2 workload, from one ncu
# capture of dram__bytes_read.sum + dram__bytes_write.sum at full size.  They describe the kernels
# as they were when the counters were taken: the digest is of the kernel sources at that time,
# and once a source file has changed the figure is no longer reported.
TRAFFIC = {"csrc_sha256_16": "7af611072cdc03a9",
           "forward_tiles": 2_401_414_912 + 7_706_880,
           "gradient_tiles": 247_456_256 + 145_509_632,
           "backward_gemms": 689_683_968 + 82_744_320}


def _csrc_digest():
    """Digest of the sources that define the three tensor kernels and their launch configuration."""
    import hashlib
    h = hashlib.sha256()
    for f in ("ptx_sm100.cuh", "kd_tile_sm100.cuh", "gemm_sm100.cuh", "npd_api.cu"):
        h.update(open(os.path.join(ROOT, "paper_2605_05940_b200", "csrc", f), "rb").read())
    return h.hexdigest()[:16]


# ------------------------------------------------------------------------------------------
# helpers
# ------------------------------------------------------------------------------------------
def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16=p["bf16_tflops"], bf16_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16=1590.0, bf16_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def __exit__(self, *exc):
        if self.proc is not None:
            time.sleep(0.15)
            self.proc.terminate()
            self.thread.join(timeout=2)

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm)}


def _dist_setup(n_gpus: int):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        backend = "nccl" if torch.cuda.is_available() else "gloo"
        dist.init_process_group(backend=backend)
    return rank, world, local


def _barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def _max_over_ranks(x: float, world, device) -> float:
    if world == 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


# ------------------------------------------------------------------------------------------
# the CPU oracle leg (cpu_baseline, and --impl reference)
# ------------------------------------------------------------------------------------------
def time_oracle(batch, sample_tokens: int, grad_scale: float):
    """Oracle forward + backward + segment statistics + selection on the first
    `sample_tokens` packed tokens (whole segments are not required: the loss step is
    per token; dW is that slice's contribution).  Returns (seconds, tokens)."""
    from oracle import npd_oracle as orc
    n = min(sample_tokens, batch.T)
    H = batch.hidden[:n].float().cpu().numpy().astype(np.float64)
    W = batch.weight.float().cpu().numpy().astype(np.float64)
    Z = batch.teacher[:n].float().cpu().numpy().astype(np.float64)
    y = batch.labels[:n].cpu().numpy()
    m = batch.loss_mask[:n].cpu().numpy()
    cu = batch.cu_seqlens.cpu().numpy()
    cu = np.concatenate([cu[cu < n], [n]]).astype(np.int32)
    t0 = time.perf_counter()
    kl, ns, nt = orc.kd_token_losses(H, W, Z, y, m, batch.tau)
    orc.kd_backward(H, W, Z, m, batch.tau, grad_scale)
    st = orc.segment_stats(cu, m, y, kl, ns, nt)
    S = len(cu) - 1
    if S >= 2:
        pairs = np.arange(S // 2) * 2
        orc.delta_ifd_select(pairs, pairs + 1, st[1], st[2], st[3], 0.0, 1.0)
    return time.perf_counter() - t0, n


def run_reference(args):
    """`--impl reference`: the oracle as it stands, on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2605_05940_b200 import synth_inputs as syn
    torch.set_num_threads(os.cpu_count() or 1)
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    sample = 256
    wl = WORKLOADS[args.config]
    # the same recipe at the sample's size (the generator needs the student logits of these rows only)
    small = {"config2_1b": dict(T=sample, min_len=32, max_len=128), "config3_rows": dict(rows=1, row_len=sample),
             "config4_short": dict(T=sample), "config5_large": dict(T=sample)}[wl["make"]]
    b = getattr(syn, wl["make"])(device=dev, d=wl["d"], V=wl["V"], **small)
    gs = 1.0 / max(b.n_loss, 1)
    for _ in range(args.warmup):
        time_oracle(b, sample, gs)
    dt = sum(time_oracle(b, sample, gs)[0] for _ in range(args.steps)) / max(args.steps, 1)
    val = sample / dt
    cores = os.cpu_count() or 1
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl["name"], "T": wl["T"], "d": wl["d"], "V": wl["V"],
                   "tau": wl["tau"], "note": "CPU oracle (NumPy fp64); each step = a 256-token sample"},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"{sample} packed tokens of the workload per step, full d and V"},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def _time_e2e(B, syn, b, step, seg_out, cond, uncond, n_pairs, stream, args, world, dev, wl, topk):
    """The same step through npd_kd_fwd_bwd_host: every step copies hidden states, teacher
    logits, boundaries, mask and labels from pinned host memory and reads the per-token
    losses back, inside the timed region.  As a training loop would, the steps alternate
    between two sets of device staging buffers, each with its compute stream, and share one copy
    stream, so that the copies of one step run while the kernels of the step before are still
    busy; every step's copies and kernels lie inside the timed region."""
    pin = lambda t: t.cpu().pin_memory()
    hh, hcu, hm, hy = map(pin, (b.hidden, b.cu_seqlens, b.loss_mask, b.labels))
    hz = None if topk else pin(b.teacher)
    htk = {k2: pin(v) for k2, v in topk.items()}
    lanes = []
    for k in range(2):
        if k == 0:
            st_b, st_step, st_seg, st_stream = b, step, seg_out, stream
        else:
            st_b = syn.KDBatch(b.name, b.T, b.d, b.V, b.S, torch.empty_like(b.hidden), b.weight,
                               torch.empty_like(b.teacher), torch.empty_like(b.cu_seqlens),
                               torch.empty_like(b.loss_mask), torch.empty_like(b.labels), b.tau)
            st_b.loss_mask.copy_(b.loss_mask)      # KDStep reads the loss-token count once
            st_topk = {k2: torch.empty_like(v) for k2, v in topk.items()}
            st_step = B.KDStep(st_b, grad_chunk_cols=args.grad_chunk_cols, grad_scale=step.grad_scale, **st_topk)
            st_seg = {k2: torch.empty_like(v) for k2, v in seg_out.items()}
            st_stream = torch.cuda.Stream(device=dev)
        hkl, hns, hnt = (torch.empty(b.T).pin_memory() for _ in range(3))
        hargs = B.make_kd_args(hh, b.weight, hz, cu_seqlens=hcu, loss_mask=hm, labels=hy, kl=hkl,
                               nll_student=hns, nll_teacher=None if topk else hnt, temperature=b.tau, **htk)
        lanes.append((st_b, st_step, st_seg, st_stream, hargs, (hkl, hns, hnt)))
    steps = max(4, min(args.steps, 10))
    copy_stream = torch.cuda.Stream(device=dev)

    def one(i):
        sb, sstep, sseg, sstream, hargs, _ = lanes[i % 2]
        B.npd_kd_fwd_bwd_host_streams(hargs, sstep.args, copy_stream, sstream)
        B.npd_segment_stats(sb.cu_seqlens, sb.loss_mask, sb.labels, sstep.kl, sstep.nll_student,
                            sstep.nll_teacher, stream=sstream, **sseg)
        if n_pairs > 0:
            B.npd_select(cond, uncond, sseg["nll_s_sum"], sseg["nll_t_sum"], sseg["count"],
                         0.0, 1.0, stream=sstream)

    one(0)
    one(1)
    # the library copies only the rows of tokens that carry loss; it reports what it copied
    h2d, d2h = B.npd_last_copy_bytes()
    torch.cuda.synchronize()
    assert lanes[1][1].status(lanes[1][3]) == B.NPD_OK
    _barrier(world)
    s0, s1 = lanes[0][3], lanes[1][3]
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    join = torch.cuda.Event()
    f0.record(s0)
    s1.wait_event(f0)
    copy_stream.wait_event(f0)
    for i in range(steps):
        one(i)
    join.record(s1)
    s0.wait_event(join)
    f1.record(s0)
    torch.cuda.synchronize()
    ms = _max_over_ranks(f0.elapsed_time(f1), world, dev) / steps
    return {"value": world * wl["T"] / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": steps,
            "note": "two staging sets and one copy stream: a step's copies overlap the previous step's kernels"}


# ------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------
def _make_batch(syn, wl, args, dev, rank):
    """The seeded synthetic batch of a configuration (every rank draws its own: replicas)."""
    kw = dict(device=dev, seed_base=wl["seed_base"] + 100 * rank)
    if wl is WORKLOADS["c2"]:
        kw.update(T=args.T or wl["T"], d=args.d or wl["d"], V=args.V or wl["V"])
    elif args.T or args.d or args.V:
        raise SystemExit("--T / --d / --V only resize the c2 workload")
    return getattr(syn, wl["make"])(**kw), kw["seed_base"]


def _input_digests(b):
    """SHA-256 of every input tensor (read back slab by slab), so that a run can be tied to its data."""
    import hashlib
    out = {}
    for name in ("hidden", "weight", "teacher", "cu_seqlens", "loss_mask", "labels"):
        t = getattr(b, name)
        h = hashlib.sha256()
        rows = max(1, (256 << 20) // max(1, t[0].numel() * t.element_size())) if t.dim() > 1 else t.numel()
        for r0 in range(0, t.shape[0], rows):
            h.update(t[r0:r0 + rows].contiguous().view(torch.uint8).cpu().numpy().tobytes())
        out[name] = h.hexdigest()[:16]
    return out


def _timed_loop(one_step, steps, stream, local, world, dev, per_step=None):
    """K steps back to back on `stream`, device-timed, clocks sampled meanwhile.  A run during
    which the GPU reported a hardware or thermal slowdown is taken again, once."""
    remeasured = False
    for attempt in range(2):
        _barrier(world)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with ClockSampler(local) as clk:
            e0.record(stream)
            for k in range(steps):
                one_step(k)
            e1.record(stream)
            stream.synchronize()
        torch.cuda.synchronize()
        _barrier(world)
        bad = {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"} & set(clk.summary()["reasons"])
        bad_any = _max_over_ranks(1.0 if bad else 0.0, world, dev) > 0
        if not bad_any or attempt == 1:
            break
        remeasured = True
        time.sleep(5.0)
    ms = _max_over_ranks(e0.elapsed_time(e1), world, dev) / steps
    return ms, dict(clk.summary(), remeasured_after_slowdown=remeasured)


def run_ours(args):
    rank, world, local = _dist_setup(args.gpus)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    from paper_2605_05940_b200 import binding as B, build as npd_build, synth_inputs as syn
    # one rank per node (re)builds the library if it is stale; the others wait for it
    if local == 0:
        npd_build.build()
    _barrier(world)

    wl = WORKLOADS[args.config]
    if wl["name"] == "c5_large_step" and torch.cuda.mem_get_info()[0] < 40 * 2**30:
        raise SystemExit("c5 needs about 30 GB of free device memory")
    b, seed_base = _make_batch(syn, wl, args, dev, rank)
    wl = dict(wl, T=b.T, d=b.d, V=b.V)
    topk = {}
    if args.teacher == "topk":     # the paper's storage form (k = 10); not the headline workload
        v, i = b.teacher.float().topk(10, dim=1)
        topk = dict(topk_values=v.contiguous(), topk_indices=i.to(torch.int32).contiguous())
    flags = B.NPD_KD_SERIALIZE_LAUNCHES if args.serialize_launches else 0
    step = B.KDStep(b, grad_chunk_cols=args.grad_chunk_cols, flags=flags, **topk)
    S = b.S
    # samples for the selection: the workload's own (prompt+answer, answer) pairs, else neighbours
    if b.cond_seg is not None:
        cond, uncond = b.cond_seg, b.uncond_seg
    else:
        cond = torch.arange(S // 2, dtype=torch.int32, device=dev) * 2
        uncond = cond + 1
    n_pairs = cond.numel()
    seg_out = dict(kl_sum=torch.empty(S, device=dev), nll_s_sum=torch.empty(S, device=dev),
                   nll_t_sum=torch.empty(S, device=dev), count=torch.empty(S, dtype=torch.int32, device=dev),
                   seg_id=torch.empty(b.T, dtype=torch.int32, device=dev))
    stream = torch.cuda.Stream(device=dev)

    if args.teacher == "topk":
        # k stored logits do not give the teacher's likelihood of a label: the selection statistics
        # (which need it) belong to the dense-teacher scoring pass and are left out here
        n_pairs = 0
        seg_out.pop("nll_t_sum")

    def tail_of_step():
        B.npd_segment_stats(b.cu_seqlens, b.loss_mask, b.labels, step.kl, step.nll_student,
                            step.nll_teacher, stream=stream, **seg_out)
        if n_pairs > 0:
            B.npd_select(cond, uncond, seg_out["nll_s_sum"], seg_out["nll_t_sum"], seg_out["count"],
                         0.0, 1.0, stream=stream)

    def one_step(_k=0):
        step.run(stream)
        tail_of_step()

    names = step.phase_names()
    with torch.cuda.stream(stream):
        for _ in range(args.warmup):
            one_step()
        launches_per_step = B.npd_last_launch_count() + 1 + (1 if n_pairs > 0 else 0)
        stream.synchronize()
        assert step.status(stream) == B.NPD_OK

        # ---- timed region: K steps, device-timed on the launching stream ----
        ms_step, clocks = _timed_loop(one_step, args.steps, stream, local, world, dev)
        tokens_per_s = world * wl["T"] / (ms_step * 1e-3)

        # ---- the same loop once more with the library's phase events attached: per-kernel times
        # under the same sustained load and clocks as the timed loop (an event between two
        # kernels also keeps the second from starting under the first one's tail, so this loop
        # can only be slower than the timed one) ----
        P = min(args.steps, 50)
        evs = [step.new_phase_events(stream) for _ in range(P)]
        stream.synchronize()

        def phase_step(k):
            step.run_recording(evs[k], stream)
            tail_of_step()

        ms_phase_loop, clocks_phase = _timed_loop(phase_step, P, stream, local, world, dev)
        per_kind = {}
        for k in range(P):
            for i, name in enumerate(names):
                per_kind[name] = per_kind.get(name, 0.0) + evs[k][i].elapsed_time(evs[k][i + 1]) / P
        groups, chunks = B.npd_phase_count(step.args)

    # ---- end to end through the host-buffer entry point ----
    e2e = None
    teacher_bytes = b.teacher.numel() * b.teacher.element_size()
    if not args.no_e2e and teacher_bytes <= 6 * 2**30:
        e2e = _time_e2e(B, syn, b, step, seg_out, cond, uncond, n_pairs, stream, args, world, dev, wl, topk)
    elif not args.no_e2e:
        e2e = {"value": None, "unit": UNIT, "note": "skipped: the pinned host copy of this workload's teacher "
               "logits (%.1f GB, twice) is not staged" % (teacher_bytes / 1e9)}

    if rank != 0:
        return
    peaks = _peaks()
    T, d, V = wl["T"], wl["d"], wl["V"]
    # Tokens without loss (the masked prompts) have zero loss and zero gradient, and the library
    # computes nothing for them (it works on the compacted loss tokens).  So the work the method
    # defines is counted on the tokens that carry loss.
    T_loss = b.n_loss
    tdv2 = 2.0 * T_loss * d * V
    rows128 = -(-T_loss // 128) * 128
    # dominant kernel = the launch group with the largest share of the step
    dom = max(per_kind, key=per_kind.get)
    dom_ms = per_kind[dom]
    # algorithmic FLOPs per step of each tensor launch group: the forward and gradient tiles each
    # form the logits once (2*T_loss*d*V); the backward launch holds both contractions (dW and dH)
    flops_of = {"forward_tiles": tdv2, "gradient_tiles": tdv2, "backward_gemms": 2 * tdv2}
    dom_flops = flops_of.get(dom, 0.0)
    achieved = dom_flops / (dom_ms * 1e-3) / 1e12
    peak_tf = peaks["bf16_sustained"]      # the kernel is timed inside a long step
    phase_sum = sum(per_kind.values())
    consistent = abs(phase_sum - ms_phase_loop) <= 0.02 * ms_phase_loop and ms_phase_loop <= 1.05 * ms_step
    mhz = clocks_phase.get("sm_mhz") or 0.0
    # Tensor-pipe utilisation at the clock the loop actually ran at: FLOPs the kernel executes (rows
    # padded to blocks of 128) over what 148 SMs x 8192 dense bf16 FLOP per clock (one 128x256x16
    # MMA per 128 clocks) could do in the measured time at the measured median clock.
    pipe = {}
    for name, fl in flops_of.items():
        if name in per_kind and mhz:
            pipe[name] = (fl * rows128 / max(T_loss, 1)) / (per_kind[name] * 1e-3 * mhz * 1e6 * 148 * 8192)
    step_flops_alg = 3 * tdv2              # 6*T_loss*d*V: the contractions the method defines
    default_case = (args.config == "c2" and T == WORKLOAD["T"] and d == WORKLOAD["d"] and V == WORKLOAD["V"]
                    and args.grad_chunk_cols == 0 and args.teacher == "dense" and not args.serialize_launches)
    traffic = TRAFFIC.get(dom) if default_case and _csrc_digest() == TRAFFIC["csrc_sha256_16"] else None
    launches_dom = chunks if dom in ("gradient_tiles", "backward_gemms") else 1
    tf_alg = step_flops_alg / (ms_step * 1e-3) / 1e12
    line = {
        "metric": METRIC, "value": tokens_per_s, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": wl["name"], "T": T, "d": d, "V": V, "tau": wl["tau"], "segments": S,
                   "loss_tokens": T_loss, "parallelism": f"replicas x{world}",
                   "l2": "inputs larger than L2 (teacher logits %.2f GB per step)" % (teacher_bytes / 1e9),
                   "grad_chunks": chunks, "teacher": args.teacher,
                   "launches": "serialised" if args.serialize_launches else "programmatic dependent",
                   "seed_base": seed_base,
                   "inputs_sha256_16": None if args.no_digests else _input_digests(b)},
        "clocks": clocks,
        "gpu_launches": launches_per_step * args.steps,
        "e2e": e2e,
        "roofline": {"bound": "tensor", "kernel": dom,
                     "achieved": achieved if consistent else None, "peak": peak_tf,
                     "unit": "TFLOP/s", "frac": achieved / peak_tf if consistent else None,
                     "frac_of_burst_peak": achieved / peaks["bf16"] if consistent else None,
                     "traffic": traffic,
                     "traffic_note": "DRAM bytes per launch (ncu, full size); launches per step: %d" % launches_dom,
                     "peak_source": f"{peaks['source']} cuBLAS bf16, sustained (kernel timed inside the loop)",
                     "kernel_ms_per_step": dom_ms, "kernel_flops_per_step": dom_flops,
                     "flops_counted_on": "tokens that carry loss",
                     "timed_in": "a loop of %d steps with phase events, clocks sampled: %s MHz median" % (P, mhz),
                     "phase_loop_ms_per_step": ms_phase_loop, "phase_sum_ms": phase_sum,
                     "null_reason": None if consistent else
                     "phase times do not add up to the step (sum %.3f ms, phase loop %.3f ms, timed loop %.3f ms)"
                     % (phase_sum, ms_phase_loop, ms_step)},
        "step_roofline": {"algorithmic_flops": step_flops_alg, "executed_flops_lower_bound": 4 * tdv2,
                          "tflops_algorithmic_per_gpu": tf_alg,
                          "frac_of_burst_peak": tf_alg / peaks["bf16"],
                          "frac_of_sustained_peak": tf_alg / peaks["bf16_sustained"],
                          "frac_of_nominal_2250": tf_alg / 2250.0,
                          "target": "0.60 of the burst peak on algorithmic FLOPs",
                          "packed_tokens_equivalent_frac_of_burst_peak":
                              3 * 2.0 * T * d * V / (ms_step * 1e-3) / 1e12 / peaks["bf16"],
                          "hbm_bound_ms": (2.0 * T * V + 2.0 * V * d) / (peaks["hbm_gbs"] * 1e9) * 1e3},
        "phase_ms": per_kind,
        "phase_mcycles": {k: v * mhz / 1e3 for k, v in per_kind.items()} if mhz else None,
        "phase_clocks": clocks_phase,
        "tensor_pipe_frac_at_loop_clock": pipe,
    }
    if not args.no_cpu_baseline and world == 1:
        sample = 1024
        sec, n = time_oracle(b, sample, step.grad_scale)
        line["cpu_baseline"] = {"value": n / sec, "unit": UNIT, "cores": os.cpu_count() or 1, "kind": "oracle",
                                "sample": f"rate on the first {n} packed tokens of the same batch (full d and V, "
                                          f"forward+backward+statistics, {sec:.1f} s); the rest of the batch was "
                                          f"not run"}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="c2", choices=sorted(WORKLOADS),
                    help="c2 = the headline workload; c3-c5 = the other full-size shapes")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--no-digests", action="store_true", help="skip hashing the inputs (profiling runs)")
    ap.add_argument("--T", type=int, default=0,
                    help="packed tokens of c2; anything but the default is a profiling case, not a bench value")
    ap.add_argument("--d", type=int, default=0, help="hidden size of c2; as for --T")
    ap.add_argument("--V", type=int, default=0, help="vocabulary size of c2; as for --T")
    ap.add_argument("--grad-chunk-cols", type=int, default=0, help="0 = library default")
    ap.add_argument("--serialize-launches", action="store_true",
                    help="launch every kernel fully serialised (comparison runs)")
    ap.add_argument("--teacher", default="dense", choices=["dense", "topk"],
                    help="dense = the benchmark's workload; topk = k=10 stored logits")
    args = ap.parse_args()
    if args.steps < 1 or args.warmup < 0:
        raise SystemExit("--steps must be at least 1")
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)
    if int(os.environ.get("WORLD_SIZE", "1")) > 1:
        import torch.distributed as dist
        if dist.is_initialized():
            dist.destroy_process_group()


if __name__ == "__main__":
    main()
