#!/usr/bin/env python
"""Benchmark of the fused packed KD forward+backward step (one JSON line).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A step is one pass of the whole hot path over one synthetic batch of the ~1B-student
workload (T=8192 packed tokens, d=1536, V=151,936, bf16, tau=1): LM-head tiles with
online softmax, per-token merge, gradient tiles, dW and dH contractions, then the
segment reductions and the Delta-IFD selection.  `value` is packed tokens/s with the
inputs resident in HBM; `e2e` is the same step through the host-buffer entry point
(host->device copies of hidden states, teacher logits, boundaries, mask and labels and
the device->host read of the per-token losses inside the timed region).

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

WORKLOAD = dict(name="c2_1b_student", T=8192, d=1536, V=151_936, tau=1.0)
METRIC = "packed tokens/sec, fused KD fwd+bwd"
UNIT = "tokens/s"


# DRAM bytes (read + write) of one launch of each tensor kernel on the c2 workload, from one ncu
# capture of dram__bytes_read.sum + dram__bytes_write.sum at full size.  They describe the kernels
# as they were when the counters were taken: the digest is of the kernel sources at that time,
# and once a source file has changed the figure is no longer reported.
TRAFFIC = {"csrc_sha256_16": "48a90c1ae0eb9b89",
           "forward_tiles": 2_371_379_712 + 7_759_104,
           "gradient_tiles": 249_105_664 + 145_410_048,
           "backward_gemms": 1_027_929_856 + 81_700_352}


def _csrc_digest():
    import glob
    import hashlib
    h = hashlib.sha256()
    for f in sorted(glob.glob(os.path.join(ROOT, "paper_2605_05940_b200", "csrc", "*"))):
        h.update(open(f, "rb").read())
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
    # the generator needs the student logits of the sampled rows only
    b = syn.config2_1b(device=dev, T=sample, d=WORKLOAD["d"], V=WORKLOAD["V"], min_len=32, max_len=128)
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
        "config": {"workload": WORKLOAD["name"], "T": WORKLOAD["T"], "d": WORKLOAD["d"], "V": WORKLOAD["V"],
                   "tau": WORKLOAD["tau"], "note": "CPU oracle (NumPy fp64); each step = a 256-token sample"},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"{sample} packed tokens of the workload per step, full d and V"},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def _time_e2e(B, syn, b, step, seg_out, pairs, n_pairs, stream, args, world, dev, wl, topk):
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
            B.npd_select(pairs, pairs + 1, sseg["nll_s_sum"], sseg["nll_t_sum"], sseg["count"],
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

    wl = dict(WORKLOAD, T=args.T, d=args.d)
    # every rank draws its own batch (independent replicas)
    b = syn.config2_1b(device=dev, T=wl["T"], d=wl["d"], V=wl["V"], seed_base=2000 + 100 * rank)
    topk = {}
    if args.teacher == "topk":     # the paper's storage form (k = 10); not the headline workload
        v, i = b.teacher.float().topk(10, dim=1)
        topk = dict(topk_values=v.contiguous(), topk_indices=i.to(torch.int32).contiguous())
    step = B.KDStep(b, grad_chunk_cols=args.grad_chunk_cols, **topk)
    S = b.S
    n_pairs = S // 2
    pairs = torch.arange(n_pairs, dtype=torch.int32, device=dev) * 2
    seg_out = dict(kl_sum=torch.empty(S, device=dev), nll_s_sum=torch.empty(S, device=dev),
                   nll_t_sum=torch.empty(S, device=dev), count=torch.empty(S, dtype=torch.int32, device=dev),
                   seg_id=torch.empty(b.T, dtype=torch.int32, device=dev))
    stream = torch.cuda.Stream(device=dev)

    if args.teacher == "topk":
        # k stored logits do not give the teacher's likelihood of a label: the selection statistics
        # (which need it) belong to the dense-teacher scoring pass and are left out here
        n_pairs = 0
        seg_out.pop("nll_t_sum")

    def one_step():
        step.run(stream)
        B.npd_segment_stats(b.cu_seqlens, b.loss_mask, b.labels, step.kl, step.nll_student,
                            step.nll_teacher, stream=stream, **seg_out)
        if n_pairs > 0:
            B.npd_select(pairs, pairs + 1, seg_out["nll_s_sum"], seg_out["nll_t_sum"], seg_out["count"],
                         0.0, 1.0, stream=stream)

    launches_per_step = None
    with torch.cuda.stream(stream):
        for _ in range(args.warmup):
            one_step()
        launches_per_step = B.npd_last_launch_count() + 1 + (1 if n_pairs > 0 else 0)
        stream.synchronize()
        assert step.status(stream) == B.NPD_OK

        # ---- timed region: K steps, device-timed on the launching stream ----
        # A run during which the GPU reported a hardware or thermal slowdown is taken again, once.
        remeasured = False
        for attempt in range(2):
            _barrier(world)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            with ClockSampler(local) as clk:
                e0.record(stream)
                for _ in range(args.steps):
                    one_step()
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
        ms_total = _max_over_ranks(e0.elapsed_time(e1), world, dev)
        ms_step = ms_total / args.steps
        tokens_per_s = world * wl["T"] / (ms_step * 1e-3)

        # ---- per-kernel times of one step (phase events recorded by the library) ----
        phase = {}
        for _ in range(3):
            for name, ms in step.run_with_phase_times(stream):
                phase.setdefault(name, []).append(ms)
        groups, chunks = B.npd_phase_count(step.args)
        per_kind = {k: sum(v) / 3 for k, v in phase.items()}           # ms per step, summed over chunks

    # ---- end to end through the host-buffer entry point ----
    e2e = None
    if not args.no_e2e:
        e2e = _time_e2e(B, syn, b, step, seg_out, pairs, n_pairs, stream, args, world, dev, wl, topk)

    if rank != 0:
        return
    peaks = _peaks()
    T, d, V = wl["T"], wl["d"], wl["V"]
    # Tokens without loss (the masked prompts) have zero loss and zero gradient, and the library
    # computes nothing for them (it works on the compacted loss tokens).  So the work the method
    # defines is counted on the tokens that carry loss.
    T_loss = b.n_loss
    tdv2 = 2.0 * T_loss * d * V
    # dominant kernel = the launch group with the largest share of the step
    dom = max(per_kind, key=per_kind.get)
    dom_ms = per_kind[dom]
    # algorithmic FLOPs per step of each tensor launch group: the forward and gradient tiles each
    # form the logits once (2*T_loss*d*V); the backward launch holds both contractions (dW and dH)
    dom_flops = 2 * tdv2 if dom == "backward_gemms" else tdv2
    achieved = dom_flops / (dom_ms * 1e-3) / 1e12
    peak_tf = peaks["bf16_sustained"]      # timed inside a long step
    step_flops_alg = 3 * tdv2              # 6*T_loss*d*V: the contractions the method defines
    default_case = (T == WORKLOAD["T"] and d == WORKLOAD["d"] and args.grad_chunk_cols == 0
                    and args.teacher == "dense")
    traffic = TRAFFIC.get(dom) if default_case and _csrc_digest() == TRAFFIC["csrc_sha256_16"] else None
    launches_dom = chunks if dom in ("gradient_tiles", "backward_gemms") else 1
    tf_alg = step_flops_alg / (ms_step * 1e-3) / 1e12
    line = {
        "metric": METRIC, "value": tokens_per_s, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": wl["name"], "T": T, "d": d, "V": V, "tau": wl["tau"], "segments": S,
                   "loss_tokens": T_loss, "parallelism": f"replicas x{world}",
                   "l2": "inputs larger than L2 (teacher logits 2.49 GB per step)",
                   "grad_chunks": chunks, "teacher": args.teacher},
        "clocks": dict(clk.summary(), remeasured_after_slowdown=remeasured),
        "gpu_launches": launches_per_step * args.steps,
        "e2e": e2e,
        "roofline": {"bound": "tensor", "kernel": dom, "achieved": achieved, "peak": peak_tf,
                     "unit": "TFLOP/s", "frac": achieved / peak_tf, "traffic": traffic,
                     "traffic_note": "DRAM bytes of one launch (ncu, full size); launches per step: %d" % launches_dom,
                     "peak_source": f"{peaks['source']} cuBLAS bf16, sustained",
                     "kernel_ms_per_step": dom_ms, "kernel_flops_per_step": dom_flops,
                     "flops_counted_on": "tokens that carry loss"},
        "step_roofline": {"algorithmic_flops": step_flops_alg, "executed_flops_lower_bound": 4 * tdv2,
                          "tflops_algorithmic_per_gpu": tf_alg,
                          "frac_of_burst_peak": tf_alg / peaks["bf16"],
                          "frac_of_sustained_peak": tf_alg / peaks["bf16_sustained"],
                          "packed_tokens_equivalent_frac_of_burst_peak":
                              3 * 2.0 * T * d * V / (ms_step * 1e-3) / 1e12 / peaks["bf16"],
                          "hbm_bound_ms": (2.0 * T * V + 2.0 * V * d) / (peaks["hbm_gbs"] * 1e9) * 1e3},
        "phase_ms": per_kind,
    }
    if not args.no_cpu_baseline and world == 1:
        sample = 512
        sec, n = time_oracle(b, sample, step.grad_scale)
        line["cpu_baseline"] = {"value": n / sec, "unit": UNIT, "cores": os.cpu_count() or 1, "kind": "oracle",
                                "sample": f"first {n} packed tokens of the same batch, full d and V, "
                                          f"forward+backward+statistics, {sec:.1f} s"}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--T", type=int, default=WORKLOAD["T"],
                    help="packed tokens; anything but the default is a profiling case, not a bench value")
    ap.add_argument("--d", type=int, default=WORKLOAD["d"], help="hidden size; as for --T")
    ap.add_argument("--grad-chunk-cols", type=int, default=0, help="0 = library default")
    ap.add_argument("--teacher", default="dense", choices=["dense", "topk"],
                    help="dense = the benchmark's workload; topk = k=10 stored logits")
    args = ap.parse_args()
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
