"""Benchmark of the TopLoc proof hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 70b|8b] [--impl ours|reference]

With --gpus N > 1 and no torchrun environment the script starts N ranks of itself
(torch.distributed.run, one per GPU); under torchrun it is one of the ranks.

One step = proof generation for every chunk of the batch followed by validation of every
proof against recomputed activations (honest-noise copy), i.e. one pass of the whole path.
The default workload is the Llama-3.1-70B-shaped batch: 256 sequences x 4096 tokens,
H = 8192, bf16 (17.18 GB), 32-token chunks, k = 128 -> 32768 proofs of 258 bytes.

Rank 0 prints one JSON line.  `value` counts chunks generated-and-validated per second with
the activations resident in HBM; `e2e` is the same through the host-buffer entry points
(pinned host memory, copies inside the timed region).  With N > 1 (torchrun) every rank
processes its own full batch: weak scaling, no collective on the data path.

Other modes (each prints its own JSON line): --decode-steps (incremental generation), --sweep
(k x chunk length x H x dtype), --direct (direct commitments, k = 128 .. 4096).
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

WORKLOADS = {
    # name: (sequences, tokens per sequence, hidden, chunk_len, k, seed)
    "70b": (256, 4096, 8192, 32, 128, 4),
    "8b": (64, 2048, 4096, 32, 128, 2),
    # every 4096-token prompt as ONE chunk of 33.5 M elements (selected in 64 segments and merged)
    "prompt70b": (64, 4096, 8192, 4096, 128, 6),
    # fp32 activations committed whole over the 32-bit field (2 + 4k byte proofs, fp32 thresholds)
    "70b-fp32-wide": (128, 4096, 8192, 32, 128, 7),
    # small cases of the two above: sized for profiler captures, not benchmark workloads
    "prompt8b": (16, 2048, 4096, 2048, 128, 9),
    "8b-fp32-wide": (64, 2048, 4096, 32, 128, 8),
}
WIDE_WORKLOADS = ("70b-fp32-wide", "8b-fp32-wide")
CAPTURE_ONLY_WORKLOADS = ("prompt8b", "8b-fp32-wide")
FALLBACK_HBM_GBS = 6650.0
# DRAM traffic of one toploc_select_kernel launch, from a profiler capture (not measured by this
# run): dram__bytes_read.sum + dram__bytes_write.sum of one launch on the 8B-shaped batch divided
# by that batch's activation bytes.  The kernel reads every chunk once whatever the batch, so the
# ratio carries over to the other bf16 batches.  None: no capture of the current kernel exists.
SELECT_DRAM_TRAFFIC = {
    "ratio_to_activation_bytes": 1.0148,   # (1083.005 MB read + 6.613 MB written) / 1073.742 MB
    "source": "ncu capture of one toploc_select_kernel launch on the 8B-shaped batch, scaled by activation bytes "
              "(profiles/select_kernel_8b_shape_ncu.md; selection code as of commit a7c3af5); not measured by this run",
}


def measured_hbm_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.thread.join(timeout=5)
        sm, smax, reasons = [], None, set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for row in self.rows:
            if len(row) != 6:
                continue
            try:
                sm.append(float(row[0]))
                smax = float(row[1])
            except ValueError:
                continue
            for name, val in zip(names, row[2:]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": smax,
                "reasons": sorted(reasons), "samples": len(sm)}


def reference_arm(args, rank):
    """The CPU oracle, as it stands, on the host cores: each step builds and validates the proofs
    of a bounded sample (the first sequence) of the workload."""
    if rank != 0:
        return
    import oracle
    from paper_2501_16007_b200 import synth
    S, T, H, L, k, seed = WORKLOADS[args.workload]
    wide = args.workload in WIDE_WORKLOADS
    act = synth.make_activations(1, T, H, torch.float32 if wide else torch.bfloat16, seed=seed, device="cpu",
                                 outliers="jitter" if wide else "fixed")
    noisy = act.clone() if L * H > (1 << 19) else synth.honest_noise(act, seed=seed + 1, rel=2.0 ** (-22 if wide else -8))
    host, host_noisy = synth.host_patterns(act), synth.host_patterns(noisy)
    chunks = T // L
    cores = oracle.default_threads()
    thr = {"t_exp": 8 * k // 128, "t_mean": 256.0, "t_median": 128.0} if wide else {}

    def step():
        proofs, status, idx = oracle.build_proofs(host, L, k, 1, T, threads=cores, wide=wide)
        oracle.verify_proofs(host_noisy, proofs, L, k, 1, T, gen_indices=idx, threads=cores, wide=wide, **thr)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / args.steps
    value = chunks / dt
    line = {
        "impl": "reference", "metric": "proof_chunks_per_s_generate_plus_verify", "value": value,
        "unit": "chunks/s", "n_gpus": args.gpus, "ranks_started": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "u32", "data": "synthetic",
        "config": {"workload": workload_name(args.workload), "sample": "first sequence (%d chunks) per step" % chunks},
        "cpu_baseline": {"value": value, "unit": "chunks/s", "cores": cores, "kind": "oracle",
                         "sample": "first sequence: %d chunks of %d x %d %s, build + verify" % (
                             chunks, L, H, "fp32 (32-bit field)" if wide else "bf16")},
        "e2e": {"value": value, "unit": "chunks/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def max_over_ranks(values, device, world):
    """Element-wise maximum of a list of per-rank numbers over all ranks (identity for one rank)."""
    if world <= 1:
        return list(values)
    import torch.distributed as dist
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def aggregate_rate(units_per_rank, world, seconds):
    """Whole-job throughput: every rank processed units_per_rank units, the job took `seconds`
    (the slowest rank's time)."""
    return units_per_rank * world / seconds


def workload_name(key):
    S, T, H, L, k, seed = WORKLOADS[key]
    return "%s-shaped: %d seq x %d tok, H=%d %s, L=%d, k=%d" % (
        {"70b": "Llama-3.1-70B", "8b": "Llama-3.1-8B", "prompt70b": "Llama-3.1-70B prompt chunks",
         "70b-fp32-wide": "Llama-3.1-70B", "prompt8b": "Llama-3.1-8B prompt chunks",
         "8b-fp32-wide": "Llama-3.1-8B"}[key], S, T, H,
        "fp32 over the 32-bit field" if key in WIDE_WORKLOADS else "bf16", L, k)


def start_ranks(n):
    """Replaces this process by `n` ranks of the same command line under torch.distributed.run."""
    port = os.environ.get("MASTER_PORT", str(29500 + os.getpid() % 2000))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n),
           "--master-addr", "127.0.0.1", "--master-port", port, os.path.abspath(__file__)] + sys.argv[1:]
    sys.stdout.flush()
    os.execv(sys.executable, cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", choices=sorted(WORKLOADS), default="70b",
                    help="70b is the headline batch; %s are small cases for profiler captures only"
                         % " and ".join(CAPTURE_ONLY_WORKLOADS))
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-recipes", action="store_true",
                    help="skip the extra timings of the 70B-shaped batch with the other input recipes (jittered "
                         "outliers, no outlier channels, magnitudes rising through every chunk)")
    ap.add_argument("--decode-steps", action="store_true",
                    help="time incremental proof generation (one row per sequence and step) instead of the main workload")
    ap.add_argument("--direct", action="store_true",
                    help="time direct commitments (index and value stored as they are) for k = 128 .. 4096 "
                         "instead of the main workload")
    ap.add_argument("--sweep", action="store_true",
                    help="time the parameter sweep (k x chunk length x H x dtype) instead of the main workload")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        start_ranks(args.gpus)  # does not return
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        reference_arm(args, rank)
        return

    import paper_2501_16007_b200 as tl
    from paper_2501_16007_b200 import synth
    import torch.distributed as dist

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("NCCL_DEBUG", "INFO")        # the communicator's rank count shows in the log
        os.environ.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
        dist.init_process_group("nccl", device_id=dev)

    if args.decode_steps:
        if rank == 0:
            print(json.dumps(decode_steps(tl, synth, dev)), flush=True)
        return
    if args.direct:
        if rank == 0:
            print(json.dumps(direct_commitments(tl, synth, dev, args.workload)), flush=True)
        return
    if args.sweep:
        if rank == 0:
            print(json.dumps(sweep(tl, synth, dev)), flush=True)
        return

    S, T, H, L, k, seed = WORKLOADS[args.workload]
    wide = args.workload in WIDE_WORKLOADS
    field = tl.TOPLOC_FIELD_32 if wide else tl.TOPLOC_FIELD_16
    # fp32: outlier magnitudes jittered -- exact ties at +-80 would be broken at random by any fp32 noise
    act = synth.make_activations(S, T, H, torch.float32 if wide else torch.bfloat16, seed=seed + 10007 * rank,
                                 device=dev, outliers="jitter" if wide else "fixed")
    # A prompt-sized bf16 chunk has thousands of elements tied at its largest magnitude, so the cut
    # is decided by index and any noise changes the selected set: that workload validates an exact copy.
    long_chunks = L * H > (1 << 19)
    # fp32 recomputation differs in the last mantissa bits only: relative 2^-22
    noise_rel = 2.0 ** -22 if wide else 2.0 ** -8
    recomputed = act.clone() if long_chunks else synth.honest_noise(act, seed=seed + 1, rel=noise_rel)
    lay, _ = tl.make_layout(act, L, k, S, T, field=field)
    lay_select, _ = tl.make_layout(act, L, k, S, T)   # toploc_select_topk hands out 16-bit patterns
    n = tl.toploc_num_chunks(lay)
    act_bytes = act.numel() * act.element_size()
    proofs = torch.empty((n, tl.toploc_layout_proof_bytes(lay)), dtype=torch.uint8, device=dev)
    status = torch.empty((n,), dtype=torch.uint8, device=dev)
    results = torch.empty((n, 40), dtype=torch.uint8, device=dev)
    thr = tl.default_thresholds(k, field=field)
    workspace = torch.empty(tl.toploc_workspace_bytes(lay), dtype=torch.uint8, device=dev)

    def step(ev=None):
        if ev:
            ev[0].record()
        tl.toploc_build_proofs(act, lay, proofs, status, workspace=workspace)
        if ev:
            ev[1].record()
        tl.toploc_verify_proofs(recomputed, lay, proofs, thr, results, workspace=workspace)
        if ev:
            ev[2].record()

    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        gpu_id = str(local_rank)
    # the sampler runs from before the warm-up (the same steps as the timed ones) to the end of the
    # timed region, so that a short timed region still sees the clock under this load
    sampler = ClockSampler(gpu_id)
    sampler.start()
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for i in range(args.steps):
        step(events[i])
    stop.record()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    clocks = sampler.stop()
    total_ms = start.elapsed_time(stop)
    build_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in events]))
    verify_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in events]))
    total_ms, build_ms, verify_ms = max_over_ranks([total_ms, build_ms, verify_ms], dev, world)
    ms_per_step = total_ms / args.steps

    # the dominant kernel on its own: toploc_select_kernel through toploc_select_topk, CUDA events
    sel_idx = torch.empty((n, k), dtype=torch.int32, device=dev)
    sel_pat = torch.empty((n, k), dtype=torch.int16, device=dev)
    sel_steps = min(args.steps, 20)
    for _ in range(3):
        tl.toploc_select_topk(recomputed, lay_select, sel_idx, sel_pat, status, workspace=workspace)
    torch.cuda.synchronize()
    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s0.record()
    for _ in range(sel_steps):
        tl.toploc_select_topk(recomputed, lay_select, sel_idx, sel_pat, status, workspace=workspace)
    s1.record()
    torch.cuda.synchronize()
    select_ms = max_over_ranks([s0.elapsed_time(s1) / sel_steps], dev, world)[0]

    accepted = int(results.cpu().numpy().view(tl.RESULT_DTYPE)["accept"].sum())
    bad_status = int(status.count_nonzero().item())

    # end to end through the host-buffer entry points (pinned memory, copies timed)
    e2e = None
    if not args.no_e2e:
        e2e = measure_e2e(tl, act, lay, n, k, thr, dev, args.e2e_steps, world)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_hbm_peak()
    select_gbs = act_bytes / (select_ms * 1e-3) / 1e9
    build_gbs = act_bytes / (build_ms * 1e-3) / 1e9
    verify_gbs = act_bytes / (verify_ms * 1e-3) / 1e9
    line = {
        "metric": "proof_chunks_per_s_generate_plus_verify",
        "value": aggregate_rate(n, world, ms_per_step * 1e-3), "unit": "chunks/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "u32", "data": "synthetic",
        "config": {"workload": workload_name(args.workload), "chunks": n, "proof_bytes": proofs.shape[1],
                   "activation_bytes": act_bytes, "l2": "inputs larger than L2 (no flush needed)",
                   "recomputed": "exact copy" if long_chunks else "honest reorder noise, relative 2^%d" % (-22 if wide else -8),
                   "outliers": "jittered magnitudes" if wide else "+-80 on fixed channels",
                   "parallelism": "chunks sharded, no collective"},
        "generate": {"ms": build_ms, "chunks_per_s": n / (build_ms * 1e-3), "GB_per_s": build_gbs,
                     "frac_of_measured_copy_peak": build_gbs / peak, "frac_of_8TBs_nominal": build_gbs / 8000.0},
        "verify": {"ms": verify_ms, "chunks_per_s": n / (verify_ms * 1e-3), "GB_per_s": verify_gbs,
                   "frac_of_measured_copy_peak": verify_gbs / peak, "frac_of_8TBs_nominal": verify_gbs / 8000.0},
        "activation_GB_per_s": 2 * act_bytes / (ms_per_step * 1e-3) / 1e9,
        # dominant kernel (87 % of the library's GPU time): algorithmic bytes = the activations, once
        "roofline": {"bound": "hbm", "kernel": "toploc_select_kernel<%s, flat>" % ("fp32" if wide else "bf16"),
                     "achieved": select_gbs, "peak": peak, "peak_kind": peak_kind + " (torch copy, burst)",
                     "unit": "GB/s", "frac": select_gbs / peak, "ms_per_launch": select_ms,
                     "algorithmic_bytes_per_launch": act_bytes,
                     "traffic": (None if wide or SELECT_DRAM_TRAFFIC["ratio_to_activation_bytes"] is None
                                 else int(act_bytes * SELECT_DRAM_TRAFFIC["ratio_to_activation_bytes"])),
                     "traffic_source": None if wide else SELECT_DRAM_TRAFFIC["source"],
                     "frac_of_8TBs_nominal": select_gbs / 8000.0},
        "roofline_calls": {"generate_frac_of_peak": build_gbs / peak, "verify_frac_of_peak": verify_gbs / peak,
                           "note": "whole calls: generate = select + interpolate kernels, verify = one kernel"},
        # build: select + interpolate, verify: one kernel; long chunks add a merge kernel to each call
        "gpu_launches": (5 * args.steps + 2 * sel_steps) if long_chunks else (3 * args.steps + sel_steps),
        "clocks": clocks,
        "checks": {"accepted_chunks": accepted, "chunks_with_status": bad_status},
        "e2e": e2e,
    }
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline(act, recomputed, S, T, H, L, k, wide)
    if args.workload == "70b" and world == 1 and not args.no_recipes:
        # The literal +-80 recipe is the streaming filter's best case (every chunk's top-128 is its
        # first 128 outliers, known after the first rows).  The same batch shape with jittered
        # outlier magnitudes, with no outlier channels, and with magnitudes that grow fourfold over every
        # chunk (the running threshold rises to the end), regenerated in place and timed the same way.
        line["other_recipes"] = {
            name: time_recipe(tl, synth, name, act, recomputed, lay, proofs, status, results, thr, workspace,
                              S, T, H, seed, min(args.steps, 20), n)
            for name in ("jitter", "none", "rising")}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def time_recipe(tl, synth, outliers, act, recomputed, lay, proofs, status, results, thr, workspace, S, T, H, seed,
                steps, n):
    """Regenerates the batch in place with another outlier recipe and times generate and verify calls
    (CUDA events, mean over `steps` steps after three warm-ups)."""
    synth.make_activations(S, T, H, act.dtype, seed=seed + 500, device=act.device, outliers=outliers, out=act)
    recomputed.copy_(synth.honest_noise(act, seed=seed + 501))
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
    for i in range(-3, steps):
        if i >= 0:
            ev[i][0].record()
        tl.toploc_build_proofs(act, lay, proofs, status, workspace=workspace)
        if i >= 0:
            ev[i][1].record()
        tl.toploc_verify_proofs(recomputed, lay, proofs, thr, results, workspace=workspace)
        if i >= 0:
            ev[i][2].record()
    torch.cuda.synchronize()
    g = float(np.mean([e[0].elapsed_time(e[1]) for e in ev]))
    v = float(np.mean([e[1].elapsed_time(e[2]) for e in ev]))
    nbytes = act.numel() * act.element_size()
    return {"generate_ms": g, "verify_ms": v, "generate_frac_of_8TBs_nominal": nbytes / g / 1e6 / 8000.0,
            "verify_frac_of_8TBs_nominal": nbytes / v / 1e6 / 8000.0,
            "accepted_chunks": int(results.cpu().numpy().view(tl.RESULT_DTYPE)["accept"].sum()), "chunks": n}


def decode_steps(tl, synth, dev, reps=20):
    """Incremental proof generation as a decoder would drive it: 256 sequences, H = 8192 bf16, one new
    row per sequence and step, a proof per 32 steps.  Times (CUDA events) of one append, of the finish,
    and of a whole 32-token interval, beside toploc_build_proofs over the same 256 assembled chunks."""
    S, L, H, k = 256, 32, 8192, 128
    act = synth.make_activations(S, L, H, torch.bfloat16, seed=11, device=dev)
    by_seq = act.view(S, L, H)
    steps = [by_seq[:, t, :].contiguous() for t in range(L)]     # the decoder's per-step outputs
    lay, _ = tl.make_layout(steps[0], L, k, S, 1)
    state = torch.empty(tl.toploc_stream_state_bytes(lay), dtype=torch.uint8, device=dev)
    ws = torch.empty(tl.toploc_stream_workspace_bytes(lay), dtype=torch.uint8, device=dev)
    proofs = torch.empty((S, tl.toploc_layout_proof_bytes(lay)), dtype=torch.uint8, device=dev)
    status = torch.empty((S,), dtype=torch.uint8, device=dev)

    def interval(ev=None):
        tl.toploc_stream_begin(state, lay)
        for t in range(L):
            tl.toploc_stream_append(steps[t], lay, t, state)
        if ev:
            ev[0].record()
        tl.toploc_stream_finish(state, lay, proofs, status, workspace=ws)
        if ev:
            ev[1].record()

    for _ in range(3):
        interval()
    torch.cuda.synchronize()
    marks = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(reps)]
    for m in marks:
        m[2].record()
        interval(m)
    torch.cuda.synchronize()
    whole = float(np.mean([m[2].elapsed_time(m[1]) for m in marks]))
    finish = float(np.mean([m[0].elapsed_time(m[1]) for m in marks]))
    blay, _ = tl.make_layout(act, L, k, S, L)
    bws = torch.empty(tl.toploc_workspace_bytes(blay), dtype=torch.uint8, device=dev)
    ref_proofs = torch.empty_like(proofs)
    for _ in range(3):
        tl.toploc_build_proofs(act, blay, ref_proofs, status, workspace=bws)
    torch.cuda.synchronize()
    b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    b0.record()
    for _ in range(reps):
        tl.toploc_build_proofs(act, blay, ref_proofs, status, workspace=bws)
    b1.record()
    torch.cuda.synchronize()
    # The producer-side hook: the final RMSNorm of the decode step, alone, and with the commitment
    # taken from its output tile while that is still in shared memory (toploc_rmsnorm_append).
    weight = torch.ones(H, dtype=torch.bfloat16, device=dev)
    y = torch.empty_like(steps[0])

    def timed_steps(fn):
        """Mean time of one decode step over whole 32-token intervals (each starts an empty chunk)."""
        def interval_of(fn):
            tl.toploc_stream_begin(state, lay)
            for t in range(L):
                fn(t)
        interval_of(fn)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            interval_of(fn)
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / (reps * L) * 1e3

    norm_alone = timed_steps(lambda t: tl.toploc_rmsnorm_append(steps[t], weight, 1e-5, lay, t, y, None))
    norm_fused = timed_steps(lambda t: tl.toploc_rmsnorm_append(steps[t], weight, 1e-5, lay, t, y, state))

    def norm_then_append(t):
        tl.toploc_rmsnorm_append(steps[t], weight, 1e-5, lay, t, y, None)
        tl.toploc_stream_append(y, lay, t, state)

    norm_separate = timed_steps(norm_then_append)
    return {"metric": "incremental_proof_generation", "sequences": S, "hidden": H, "interval_tokens": L, "k": k,
            "us_per_append": (whole - finish) / L * 1e3, "us_finish": finish * 1e3, "us_per_interval": whole * 1e3,
            "us_batch_build_of_the_same_chunks": b0.elapsed_time(b1) / reps * 1e3,
            "bytes_per_append": S * H * 2, "identical_to_batch": bool(torch.equal(proofs, ref_proofs)),
            "final_norm": {"us_norm_alone": norm_alone, "us_norm_with_fused_commit": norm_fused,
                           "us_norm_then_separate_append": norm_separate,
                           "us_added_by_fused_commit": norm_fused - norm_alone,
                           "us_added_by_separate_append": norm_separate - norm_alone}}


def direct_commitments(tl, synth, dev, workload, reps=10):
    """toploc_commit_direct / toploc_verify_direct over the workload's batch for k = 128 .. 4096:
    CUDA-event time per call, activation GB/s (the batch's bytes, once) and its fraction of the
    measured copy peak."""
    S, T, H, L, _, seed = WORKLOADS[workload]
    dtype = torch.float32 if workload in WIDE_WORKLOADS else torch.bfloat16
    act = synth.make_activations(S, T, H, dtype, seed=seed, device=dev)
    rec = synth.honest_noise(act, seed=seed + 100)
    peak, peak_kind = measured_hbm_peak()
    nbytes = act.numel() * act.element_size()
    points = []
    for k in (128, 512, 1024, 2048, 4096):
        lay, _ = tl.make_layout(act, L, k, S, T)
        commits, status = tl.toploc_commit_direct(act, lay)
        results, dev_bins = tl.toploc_verify_direct(rec, lay, commits)
        thr = tl.default_thresholds(k)

        def timed(fn):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                fn()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / reps

        t_commit = timed(lambda: tl.toploc_commit_direct(act, lay, commits, status))
        t_verify = timed(lambda: tl.toploc_verify_direct(rec, lay, commits, thr, results, dev_bins))
        got = results.cpu().numpy().view(tl.RESULT_DTYPE).reshape(-1)
        points.append({"k": k, "commit_bytes": 6 * k, "commit_ms": t_commit, "verify_ms": t_verify,
                       "commit_GB_per_s": nbytes / t_commit / 1e6, "verify_GB_per_s": nbytes / t_verify / 1e6,
                       "commit_frac_of_peak": nbytes / t_commit / 1e6 / peak,
                       "verify_frac_of_peak": nbytes / t_verify / 1e6 / peak,
                       "accepted": int(got["accept"].sum()), "chunks": int(got.size),
                       "mean_topk_mismatch": float(got["topk_mismatch"].mean())})
    return {"metric": "direct_commitments", "workload": workload_name(workload), "activation_bytes": nbytes,
            "activations": "fp32, upper 16 bits of a pattern committed" if dtype == torch.float32 else "bf16",
            "peak_GB_per_s": peak, "peak_kind": peak_kind, "recomputed": "honest reorder noise, relative 2^-8",
            "points": points}


def sweep(tl, synth, dev, reps=5):
    """k in {32, 64, 128, 256} x chunk length in {16, 32, 64} x H in {2048, 4096, 8192} x {bf16, fp32},
    128 sequences x 1024 tokens each: generate and verify times per point (CUDA events, mean of reps)."""
    peak, peak_kind = measured_hbm_peak()
    S, T = 128, 1024
    points = []
    for dtype, name in ((torch.bfloat16, "bf16"), (torch.float32, "fp32")):
        for H in (2048, 4096, 8192):
            act = synth.make_activations(S, T, H, dtype, seed=50 + H // 1024, device=dev)
            rec = synth.honest_noise(act, seed=9)
            nbytes = act.numel() * act.element_size()
            for L in (16, 32, 64):
                for k in (32, 64, 128, 256):
                    lay, _ = tl.make_layout(act, L, k, S, T)
                    n = tl.toploc_num_chunks(lay)
                    proofs = torch.empty((n, 2 + 2 * k), dtype=torch.uint8, device=dev)
                    status = torch.empty((n,), dtype=torch.uint8, device=dev)
                    results = torch.empty((n, 40), dtype=torch.uint8, device=dev)
                    ws = torch.empty(tl.toploc_workspace_bytes(lay), dtype=torch.uint8, device=dev)
                    thr = tl.default_thresholds(k)

                    def timed(fn):
                        for _ in range(2):
                            fn()
                        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        a.record()
                        for _ in range(reps):
                            fn()
                        b.record()
                        torch.cuda.synchronize()
                        return a.elapsed_time(b) / reps

                    g = timed(lambda: tl.toploc_build_proofs(act, lay, proofs, status, workspace=ws))
                    v = timed(lambda: tl.toploc_verify_proofs(rec, lay, proofs, thr, results, workspace=ws))
                    acc = int(results.cpu().numpy().view(tl.RESULT_DTYPE)["accept"].sum())
                    points.append({"dtype": name, "H": H, "L": L, "k": k, "chunks": n,
                                   "generate_ms": round(g, 4), "verify_ms": round(v, 4),
                                   "generate_chunks_per_s": round(n / g * 1e3), "verify_chunks_per_s": round(n / v * 1e3),
                                   "generate_frac_of_peak": round(nbytes / g / 1e6 / peak, 3),
                                   "verify_frac_of_peak": round(nbytes / v / 1e6 / peak, 3), "accepted": acc})
            del act, rec
    return {"metric": "sweep", "peak_GB_per_s": peak, "peak_kind": peak_kind, "unit": "fraction of HBM peak",
            "batch": "%d sequences x %d tokens" % (S, T), "points": points}


def measure_e2e(tl, act, lay, n, k, thr, dev, steps, world):
    """Host-buffer path: activations in pinned host memory, proofs and results returned to the host."""
    import torch.distributed as dist
    act_bytes = act.numel() * act.element_size()
    try:
        h_act = torch.empty(act.shape, dtype=act.dtype, pin_memory=True)
    except RuntimeError as e:
        return {"value": None, "unit": "chunks/s", "error": "pinned allocation failed: %s" % e}
    h_act.copy_(act)
    h_proofs = torch.empty((n, tl.toploc_layout_proof_bytes(lay)), dtype=torch.uint8, pin_memory=True)
    h_status = torch.empty((n,), dtype=torch.uint8, pin_memory=True)
    h_results = torch.empty((n, 40), dtype=torch.uint8, pin_memory=True)
    staging = torch.empty(max(tl.toploc_staging_bytes(lay) * 8, 1 << 20), dtype=torch.uint8, device=dev)

    def step():
        tl.toploc_build_proofs_host(h_act, lay, h_proofs, h_status, staging)
        tl.toploc_verify_proofs_host(h_act, lay, h_proofs, thr, h_results, staging)

    step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    torch.cuda.synchronize()
    dt = (time.perf_counter() - t0) / steps
    dt = max_over_ranks([dt], dev, world)[0]
    proofs_b = n * tl.toploc_layout_proof_bytes(lay)
    return {"value": aggregate_rate(n, world, dt), "unit": "chunks/s", "ms_per_step": dt * 1e3, "steps": steps,
            "h2d_bytes_per_step": 2 * act_bytes + proofs_b, "d2h_bytes_per_step": proofs_b + n + n * 40,
            "note": "build then verify (identical copy) from pinned host memory; PCIe-bound"}


def cpu_baseline(act, recomputed, S, T, H, L, k, wide=False):
    """The oracle, as it stands, on a bounded sample of the same batch: whole sequences from the
    front, at least 1024 chunks where the batch has them (about 5 to 30 s on the host cores)."""
    import oracle
    from paper_2501_16007_b200 import synth
    per_seq = (T + L - 1) // L
    seqs = max(1, min(S, -(-1024 // per_seq))) if L * H <= (1 << 19) else 1   # a prompt-sized chunk takes seconds
    host = synth.host_patterns(act[:seqs * T])
    host_rec = synth.host_patterns(recomputed[:seqs * T])
    cores = oracle.default_threads()
    chunks = seqs * per_seq
    t0 = time.perf_counter()
    proofs, status, idx = oracle.build_proofs(host, L, k, seqs, T, threads=cores, wide=wide)
    t1 = time.perf_counter()
    oracle.verify_proofs(host_rec, proofs, L, k, seqs, T, gen_indices=idx, threads=cores, wide=wide,
                         **({"t_exp": 8 * k // 128, "t_mean": 256.0, "t_median": 128.0} if wide else {}))
    t2 = time.perf_counter()
    return {"value": chunks / (t2 - t0), "unit": "chunks/s", "cores": cores, "kind": "oracle",
            "sample": "first %d sequence(s): %d chunks of %d x %d %s, build + verify" % (
            seqs, chunks, L, H, "fp32 (32-bit field)" if wide else "bf16"),
            "generate_chunks_per_s": chunks / (t1 - t0), "verify_chunks_per_s": chunks / (t2 - t1)}


if __name__ == "__main__":
    main()
