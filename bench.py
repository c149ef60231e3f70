#!/usr/bin/env python
"""Benchmark of the draft-and-verify decision path (ssd_ctc_draft -> ssd_entropy_gate ->
ssd_verify) on synthetic logits shaped like the paper's workloads.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A step is one pass of the whole path over one ragged batch.  One JSON line is printed by rank 0:
utterances/s with the inputs resident in HBM, the same metric end to end from pinned host
buffers, the HBM roofline fraction of the streaming kernels (timed with CUDA events that the
library records around them, on at least 24 launches whatever K is), the clocks seen under load,
the CPU oracle timed on the host cores as a reported baseline, and the same figures for the
other benchmark configurations in `per_config`.  `--impl reference` times that oracle alone.
"""
import argparse
import datetime
import hashlib
import json
import math
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "utterances/s for CTC draft+gate+verify"
UNIT = "utterances/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0        # the "~8 TB/s" the metric is stated against
KERNEL_LAUNCHES = 24            # event-carrying launches per streaming kernel, after the timed region
SMALL_SET_BYTES = 2e9           # below this, three input sets are rotated so that no step finds its
                                # inputs in the 126 MB L2; above it one set is many times the L2
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "ncu_traffic.json")
KERNEL_SOURCES = ["ssd_common.cuh", "ssd_stream.cuh", "ssd_ranges.cuh", "ssd_ctc.cu", "ssd_verify.cu",
                  "ssd_api.cu"]


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=3,
                    help="workload index: 1..3 benchmark configurations (3, the largest that fits "
                         "one GPU, is the headline); 5, 6 the paper's own shape at its "
                         "high-accuracy / high-RTFx operating point")
    ap.add_argument("--e2e-steps", type=int, default=0, help="0: 3 for workloads of more than 2 GB per step, else 30")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-config", action="store_true",
                    help="leave out the per_config records (the other benchmark configurations)")
    ap.add_argument("--verify-mode", default="full", choices=["full", "early_exit"],
                    help="full: ssd_verify reads every row of every verified utterance (the "
                         "benchmark metric); early_exit: ssd_verify_early_exit in its place, a "
                         "separate mode whose line says so in config.verify_mode")
    ap.add_argument("--sweep", default=None, metavar="FILE",
                    help="time every point of the throughput sweep (configuration 4) and write one "
                         "JSON line per point to FILE instead of the benchmark line")
    ap.add_argument("--sweep-filter", default="", help="only points whose name contains this")
    ap.add_argument("--ncu-small", action="store_true",
                    help="profiling aid: one input set, no end-to-end leg, no CPU baseline, no per_config")
    ap.add_argument("--ncu-stage1", action="store_true",
                    help="profiling aid: only the CTC batch of --config (a fraction of a GB even "
                         "where the whole step holds tens), ssd_ctc_draft three times, no timing")
    ap.add_argument("--ncu-rows", type=int, default=0,
                    help="profiling aid: ssd_verify alone on this many rows of --config's LLM "
                         "vocabulary, three times, no timing")
    return ap.parse_args()


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def kernel_source_hash() -> str:
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2603_11243_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def recorded_traffic(kernel: str, units: float):
    """DRAM bytes per launch of `kernel` from the committed ncu capture, scaled by the units
    (bytes of logits) this launch processes; None when the kernels changed since the capture."""
    try:
        with open(TRAFFIC_FILE) as f:
            rec = json.load(f)
        e = rec[kernel]
        if rec.get("source_sha256") != kernel_source_hash():
            return None
        return float(e["dram_bytes_per_launch"]) * units / float(e["algorithmic_bytes_per_launch"])
    except Exception:
        return None


# ---- clocks --------------------------------------------------------------------------------
CLOCK_FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
                "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
                "clocks_event_reasons.sw_power_cap")


class ClockSampler:
    def __init__(self, device_index: int):
        import torch
        self.path = tempfile.mktemp(prefix="ssd_clocks_", suffix=".csv")
        uuid = str(torch.cuda.get_device_properties(device_index).uuid)
        if not uuid.startswith("GPU-"):
            uuid = "GPU-" + uuid
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "--id=" + uuid, "--query-gpu=" + CLOCK_FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            pass

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        rows = []
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 8:
                    continue
                try:
                    ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                    rows.append((ts, float(f[1]), float(f[2]), f[4:8]))
                except ValueError:
                    continue
            os.unlink(self.path)
        except OSError:
            pass
        return rows


def summarise_clocks(rows, windows, note):
    names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
    inside = [r for r in rows if any(a <= r[0] <= b for a, b in windows)]
    if not inside:
        return {"sm_mhz": None, "sm_max_mhz": rows[0][2] if rows else None, "reasons": [],
                "samples": 0, "note": "no nvidia-smi sample fell inside the load windows"}
    reasons = sorted({n for r in inside for n, v in zip(names, r[3]) if v == "Active"})
    return {"sm_mhz": statistics.median(r[1] for r in inside), "sm_max_mhz": inside[0][2],
            "reasons": reasons, "samples": len(inside), "note": note}


# ---- our arm ---------------------------------------------------------------------------------
def elem_size(w):
    return 2 if w.dtype == "bf16" else 4


def build_sets(w, device, n_sets, batch_lengths=None, verify_mode="full"):
    """Input sets and pre-marshalled calls.  The verify logits of a set have one row per draft
    token of the set's own CTC drafts (found by running stage 1 once, untimed).  With
    batch_lengths (a list of per-batch utterance lengths) every set is one of those batches."""
    import torch
    from paper_2603_11243_b200 import binding as ssd
    from paper_2603_11243_b200 import synth
    sets = []
    for i in range(n_sets):
        wi = synth.scaled(w, seed=w.seed + 7 * i)
        lengths = None
        if batch_lengths is not None:
            lengths = batch_lengths[i]
            wi = synth.scaled(wi, B=len(lengths))
        cb = synth.make_ctc_batch(wi, device, lengths)
        B, N = wi.B, cb.logits.shape[0]
        off = cb.frame_off.to(device)
        s1 = ssd.alloc_ctc_outputs(N, B, device)
        ssd.ssd_ctc_draft(cb.logits, off, wi.blank_id, wi.max_draft_len, out=s1)
        gate = ssd.alloc_gate_outputs(B, device)
        # the gate's first form once, as a check of the form the timed steps use
        ssd.ssd_entropy_gate(s1["frame_entropy"], off, wi.tau_ctc, out=gate)
        g2 = ssd.ssd_entropy_gate_from_maxima(s1["utt_max_entropy"], s1["utt_status"], wi.tau_ctc)
        torch.cuda.synchronize()
        assert torch.equal(g2["gate_accept"], gate["gate_accept"]), "the two forms of the gate disagree"
        K = s1["draft_len"].cpu().tolist()
        vb = synth.make_verify_batch(wi, K, device)
        M = vb.logits.shape[0]
        tok_off, ids = vb.tok_off.to(device), vb.draft_ids.to(device)
        code = ssd.BF16 if wi.dtype == "bf16" else ssd.F32
        s2 = ssd.alloc_verify_outputs(M, B, device, ssd.ssd_verify_workspace_bytes(B, M, wi.V_llm, code))
        skipped = gate["gate_accept"].cpu().numpy().astype(bool)
        m_active = int(sum(k for k, s in zip(K, skipped) if not s))
        es = elem_size(wi)
        if verify_mode == "early_exit":
            # the full call first (its decisions are the check), then the early-exit one, whose
            # rows_read give the bytes this mode really reads
            ssd.ssd_verify(vb.logits, tok_off, ids, wi.tau_slm, skip=gate["gate_accept"], out=s2)
            full_acc = s2["accepted_len"].clone()
            s2 = ssd.alloc_early_exit_outputs(M, B, wi.V_llm, code, device)
            call_verify = ssd.bind_verify_early_exit(vb.logits, tok_off, ids, wi.tau_slm, s2,
                                                     skip=gate["gate_accept"])
            call_verify()
            torch.cuda.synchronize()
            assert torch.equal(full_acc, s2["accepted_len"]), "early exit changed a decision"
            rr = s2["rows_read"]
            if bool((rr >= 0).all().item()):
                m_active = int(rr.sum().item())
        else:
            call_verify = ssd.bind_verify(vb.logits, tok_off, ids, wi.tau_slm, s2,
                                          skip=gate["gate_accept"])
        sets.append(dict(
            w=wi, cb=cb, vb=vb, off=off, tok_off=tok_off, ids=ids, s1=s1, gate=gate, s2=s2,
            B=B, N=N, M=M, K=K, m_active=m_active,
            ctc_bytes=N * wi.V_ctc * es, verify_bytes=m_active * wi.V_llm * es,
            call_ctc=ssd.bind_ctc_draft(cb.logits, off, wi.blank_id, wi.max_draft_len, s1),
            call_gate=ssd.bind_entropy_gate_from_maxima(s1["utt_max_entropy"], s1["utt_status"],
                                                        wi.tau_ctc, gate),
            call_verify=call_verify))
    return sets


def step(s, o_ctc=None, o_ver=None):
    """One pass of the path over one batch: frame statistics and collapse (Eq. 2, Section 2.1),
    the entropy gate (Eq. 3; from the utterance maxima the first call left), verification of
    the utterances the gate did not accept (Eq. 5, Section 2.3)."""
    s["call_ctc"](o_ctc)
    s["call_gate"]()
    s["call_verify"](o_ver)


def make_events(n):
    """n timing events whose CUDA handles exist (torch creates the handle at the first record)."""
    import torch
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(n)]
    for e in evs:
        e.record()
    torch.cuda.synchronize()
    return evs


def time_kernels(sets, launches=KERNEL_LAUNCHES):
    """Durations (ms) of the two streaming kernels over `launches` further steps, each step
    carrying the events the library records just around those kernels.  (An event between two
    kernels keeps the second from being scheduled early, so the steps of the timed region carry
    none.)"""
    import torch
    from paper_2603_11243_b200 import binding as ssd
    n_sets = len(sets)
    ev = make_events(4 * launches)
    for j in range(launches):
        a, b = ssd.LaunchOpts(), ssd.LaunchOpts()
        a.ev_begin, a.ev_end = ev[4 * j].cuda_event, ev[4 * j + 1].cuda_event
        b.ev_begin, b.ev_end = ev[4 * j + 2].cuda_event, ev[4 * j + 3].cuda_event
        step(sets[j % n_sets], a, b)
    torch.cuda.synchronize()
    t_ctc = [ev[4 * j].elapsed_time(ev[4 * j + 1]) for j in range(launches)]
    t_ver = [ev[4 * j + 2].elapsed_time(ev[4 * j + 3]) for j in range(launches)]
    ctc_bytes = statistics.mean(sets[j % n_sets]["ctc_bytes"] for j in range(launches))
    ver_bytes = statistics.mean(sets[j % n_sets]["verify_bytes"] for j in range(launches))
    return t_ctc, t_ver, ctc_bytes, ver_bytes


def roof(kernel, nbytes, times_ms, peak, peak_kind):
    """Roofline record of one streaming kernel: algorithmic bytes per launch over the mean
    launch duration (median and best beside it), against the measured copy bandwidth and against
    the nominal 8 TB/s."""
    times = [t for t in times_ms if t > 0]
    if not times or nbytes <= 0:
        return {"kernel": kernel, "bound": "hbm", "achieved": 0.0, "peak": peak, "unit": "GB/s",
                "frac": 0.0, "peak_kind": "of " + peak_kind, "traffic": None,
                "algorithmic_bytes_per_launch": int(nbytes), "launches_timed": len(times),
                "note": "nothing to read in this configuration"}
    avg, med, best = statistics.mean(times), statistics.median(times), min(times)
    gbs = lambda ms: nbytes / (ms * 1e-3) / 1e9
    return {"kernel": kernel, "bound": "hbm", "achieved": round(gbs(avg), 1), "peak": peak,
            "unit": "GB/s", "frac": round(gbs(avg) / peak, 4), "peak_kind": "of " + peak_kind,
            "frac_median": round(gbs(med) / peak, 4), "frac_best": round(gbs(best) / peak, 4),
            "frac_of_nominal": round(gbs(avg) / NOMINAL_HBM_GBS, 4), "nominal_peak": NOMINAL_HBM_GBS,
            "traffic": recorded_traffic(kernel, nbytes),
            "algorithmic_bytes_per_launch": int(nbytes), "launches_timed": len(times),
            "avg_launch_us": round(avg * 1e3, 2), "median_launch_us": round(med * 1e3, 2),
            "min_launch_us": round(best * 1e3, 2)}


def timed_steps(sets, K, W, barrier=None):
    """W warm-up steps, then K steps between two events with a synchronize on both sides.
    Returns (ms for the K steps, wall-clock window, kernels launched in the window)."""
    import torch
    from paper_2603_11243_b200 import binding as ssd
    n_sets = len(sets)
    for i in range(W):
        step(sets[i % n_sets])
    torch.cuda.synchronize()
    ev = make_events(2)
    if barrier:
        barrier()
    torch.cuda.synchronize()
    wall0 = time.time()
    l0 = int(ssd.lib().ssd_launch_count())
    ev[0].record()
    for i in range(K):
        step(sets[i % n_sets])
    ev[1].record()
    torch.cuda.synchronize()
    wall1 = time.time()
    launches = int(ssd.lib().ssd_launch_count()) - l0
    if barrier:
        barrier()
    return ev[0].elapsed_time(ev[1]), (wall0, wall1), launches


def sets_for(w, device, verify_mode="full", one_set=False):
    from paper_2603_11243_b200 import synth
    batch_lengths = None
    est = w.B * (0.5 * (w.t_lo + w.t_hi) * w.V_ctc + min(w.max_draft_len, 0.2 * (w.t_lo + w.t_hi)) * w.V_llm) * elem_size(w)
    n_sets = 1 if (one_set or est > SMALL_SET_BYTES) else 3
    if w.name.startswith("paper_"):
        # the paper's batching: a pool of utterances, length-sorted, <= 50,000 frames per batch
        batch_lengths = synth.length_sorted_batches(synth.draw_lengths(w))
        n_sets = 1 if one_set else len(batch_lengths)
    return build_sets(w, device, n_sets, batch_lengths, verify_mode), batch_lengths


def l2_note(sets):
    s0 = sets[0]
    per_set = s0["ctc_bytes"] + s0["M"] * s0["w"].V_llm * elem_size(s0["w"])
    if len(sets) > 1:
        return ("inputs larger than L2: %d distinct input batches of %.2f GB rotated" %
                (len(sets), per_set / 1e9))
    return "inputs larger than L2: one input batch of %.2f GB, %d times the 126 MB L2" % (
        per_set / 1e9, int(per_set / 126e6))


def workload_string(idx, base, w, batch_lengths):
    return ("configs[%s] %s: B=%s utterances per GPU, T~%s[%d,%d], V_ctc=%d, V_llm=%d, "
            "draft_len<=%d, %s logits (fp32 accumulation)" %
            (idx, base.name,
             w.B if batch_lengths is None else
             "%d in %d length-sorted batches of <=50,000 frames; a step is one batch;"
             % (w.B, len(batch_lengths)),
             w.t_dist, w.t_lo, w.t_hi, w.V_ctc, w.V_llm, w.max_draft_len, w.dtype))


PER_CONFIG = [("configs[1]", 1, None), ("configs[2]", 2, None),
              ("configs[4] B=64 V_llm=49152 bf16", 4, (64, 49152, "bf16")),
              ("configs[4] B=64 V_llm=152064 bf16", 4, (64, 152064, "bf16")),
              ("configs[4] B=64 V_llm=49152 f32", 4, (64, 49152, "f32")),
              ("configs[4] B=64 V_llm=152064 f32", 4, (64, 152064, "f32")),
              ("configs[4] B=1024 V_llm=49152 bf16", 4, (1024, 49152, "bf16")),
              ("configs[4] B=1024 V_llm=49152 f32", 4, (1024, 49152, "f32")),
              ("configs[4] B=1 V_llm=32000 bf16", 4, (1, 32000, "bf16")),
              ("configs[4] B=1 V_llm=152064 f32", 4, (1, 152064, "f32"))]


def run_per_config(device, peak, peak_kind, skip_idx, cpu=True):
    """The other benchmark configurations, each timed like the headline (fewer steps): whole-step
    throughput, both streaming kernels on KERNEL_LAUNCHES event-carrying launches, the oracle on
    a bounded sample."""
    import torch
    from paper_2603_11243_b200 import synth
    out = {}
    for name, idx, point in PER_CONFIG:
        if idx == skip_idx and point is None:
            continue
        w = synth.CONFIGS[idx] if point is None else synth.sweep_point(*point)
        t0 = time.time()
        sets, _ = sets_for(w, device)
        est_ms = max(0.02, sum(s["ctc_bytes"] + s["verify_bytes"] for s in sets) / len(sets) / 5e9)
        K = int(max(20, min(400, 60.0 / est_ms)))
        ms, _, launches = timed_steps(sets, K, 5)
        t_ctc, t_ver, ctc_b, ver_b = time_kernels(sets)
        units = sum(sets[i % len(sets)]["B"] for i in range(K))
        step_bytes = statistics.mean(s["ctc_bytes"] + s["verify_bytes"] for s in sets)
        rec = {"workload": workload_string(idx, w, w, None), "steps": K,
               "value": round(units / (ms * 1e-3), 1), "unit": UNIT,
               "ms_per_step": round(ms / K, 5), "gpu_launches_per_step": launches / K,
               "logits_bytes_per_step": int(step_bytes),
               "step_hbm_gbs": round(step_bytes / (ms / K * 1e-3) / 1e9, 1),
               "step_frac_of_peak": round(step_bytes / (ms / K * 1e-3) / 1e9 / peak, 4),
               "step_frac_of_nominal": round(step_bytes / (ms / K * 1e-3) / 1e9 / NOMINAL_HBM_GBS, 4),
               "l2": l2_note(sets),
               "roofline_ctc": roof("ctc_rows_tma", ctc_b, t_ctc, peak, peak_kind),
               "roofline_verify": roof("verify_rows_tma", ver_b, t_ver, peak, peak_kind)}
        if cpu:
            rec["cpu_baseline"] = cpu_baseline(sets[0], budget_s=2.5)
        rec["seconds_spent"] = round(time.time() - t0, 1)
        out[name] = rec
        del sets
        torch.cuda.empty_cache()
    return out


def run_ours(args):
    import torch
    from paper_2603_11243_b200 import binding as ssd
    from paper_2603_11243_b200 import build as lib_build
    from paper_2603_11243_b200 import dist as D
    from paper_2603_11243_b200 import synth

    rank, local_rank, world = D.init("nccl")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: libssd has no CPU path")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if rank == 0:
        lib_build.build()
    D.barrier()
    ssd.lib()

    base = synth.CONFIGS[args.config]
    w = synth.scaled(base, seed=D.rank_seed(base.seed, rank))
    sets, batch_lengths = sets_for(w, device, args.verify_mode, one_set=args.ncu_small)
    n_sets = len(sets)
    K, W = args.steps, args.warmup

    # ---- timed region: W warm-up steps, then K steps with the inputs resident in HBM ---------
    sampler = ClockSampler(local_rank) if rank == 0 else None
    ms_total, window, launches = timed_steps(sets, K, W, barrier=D.barrier)
    windows, clock_note = [window], "timed region"
    if rank == 0 and window[1] - window[0] < 0.6 and not args.ncu_small:
        # the region is too short for a 50 ms sampler: keep the same load up a little longer
        wall2 = time.time()
        i = 0
        while time.time() - wall2 < 0.7:
            step(sets[i % n_sets])
            i += 1
            if i % 50 == 0:
                torch.cuda.synchronize()
        torch.cuda.synchronize()
        windows.append((wall2, time.time()))
        clock_note = "timed region plus %d further untimed steps of the same load" % i
    clock_rows = sampler.stop() if sampler else []

    ms_max, units = D.reduce_max_sum(ms_total, float(sum(sets[i % n_sets]["B"] for i in range(K))),
                                     device)
    value = units / (ms_max * 1e-3)
    step_bytes = statistics.mean(sets[i % n_sets]["ctc_bytes"] + sets[i % n_sets]["verify_bytes"]
                                 for i in range(K))
    peak, peak_kind = peaks()

    # ---- the streaming kernels alone, on KERNEL_LAUNCHES further steps that carry events ------
    t_ctc, t_ver, ctc_bytes, ver_bytes = time_kernels(sets, 3 if args.ncu_small else KERNEL_LAUNCHES)
    vkern = "verify_rows_tma" if args.verify_mode == "full" else "verify_rows_ee"

    # ---- end to end: pinned host buffers in, decisions out, every step ---------------------
    e2e = None
    if not args.ncu_small:
        e2e_steps = args.e2e_steps or (3 if step_bytes > 2e9 else 30)
        e2e = run_e2e(sets[0], device, e2e_steps, D, world)

    if rank != 0:
        D.finalize()
        return
    next_rows = None if (args.ncu_small or args.verify_mode != "full") else \
        time_next_rows(sets, device, peak)
    s0 = sets[0]
    gate_acc = float(s0["gate"]["gate_accept"].float().mean().item())
    all_acc = s0["s2"]["all_accepted"].cpu().numpy().astype(bool)
    skipped = s0["gate"]["gate_accept"].cpu().numpy().astype(bool)
    r_ctc = roof("ctc_rows_tma", ctc_bytes, t_ctc, peak, peak_kind)
    r_ver = roof(vkern, ver_bytes, t_ver, peak, peak_kind)
    line = {
        "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": W, "ms_per_step": round(ms_max / K, 5), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {
            "workload": workload_string(args.config, base, w, batch_lengths),
            "logits_dtype": w.dtype, "accumulation_dtype": "f32",
            "generator": w.variant, "tau_ctc": w.tau_ctc, "tau_slm": w.tau_slm,
            "verify_mode": args.verify_mode,
            "calls_per_step": "ssd_ctc_draft, ssd_entropy_gate (from the utterance maxima), ssd_verify",
            "frames_per_step": s0["N"], "verify_rows_per_step": s0["M"],
            "verify_rows_read_per_step": s0["m_active"],
            "logits_bytes_per_step": int(step_bytes),
            "l2": l2_note(sets) + "; each step reads %.2f GB once" % (step_bytes / 1e9),
            "parallelism": "utterances sharded over %d rank(s), no data-path collective" % world},
        "gpu_launches": launches,
        # `roofline` is the kernel that holds most of the step's device time
        "roofline": r_ver if sum(t_ver) >= sum(t_ctc) else r_ctc,
        "roofline_ctc": r_ctc,
        "roofline_verify": r_ver,
        "step_hbm_gbs": round(step_bytes / (ms_max / K * 1e-3) / 1e9, 1),
        "step_frac_of_peak": round(step_bytes / (ms_max / K * 1e-3) / 1e9 / peak, 4),
        "step_frac_of_nominal": round(step_bytes / (ms_max / K * 1e-3) / 1e9 / NOMINAL_HBM_GBS, 4),
        "decisions": {"gate_accept_frac": round(gate_acc, 4),
                      "verify_all_accepted_frac_of_verified":
                          round(float(all_acc[~skipped].mean()) if (~skipped).any() else 0.0, 4)},
        "clocks": summarise_clocks(clock_rows, windows, clock_note),
        "e2e": e2e,
        "next_rows": next_rows,
    }
    if world == 1 and not args.no_cpu_baseline and not args.ncu_small:
        line["cpu_baseline"] = cpu_baseline(s0, budget_s=16.0, single_thread_too=True)
    del sets
    torch.cuda.empty_cache()
    if world == 1 and not args.ncu_small and not args.no_per_config:
        line["per_config"] = run_per_config(device, peak, peak_kind, args.config,
                                            cpu=not args.no_cpu_baseline)
    print(json.dumps(line), flush=True)
    D.finalize()


def time_next_rows(sets, device, peak):
    """The calls that follow the path (not part of `value`): the operating-point sweep over the
    step's stored maxima and log-likelihoods, the assembly of Eq. 7, and one greedy decoding
    step over as many rows as the step has utterances left to the auto-regressive pass would
    be too small to time, so over the first 1024 verify rows of each input set in turn."""
    import torch
    from paper_2603_11243_b200 import binding as ssd
    n_sets = len(sets)
    pairs = [(0.7 + 2.3 * i / 15.0, ts) for i in range(16) for ts in (0.1, 0.2)]
    tc, ts = [p[0] for p in pairs], [p[1] for p in pairs]
    R = min(1024, min(s["M"] for s in sets))
    if R == 0:
        return None
    prep = []
    for s in sets:
        sw = ssd.ssd_threshold_sweep(s["s1"]["utt_max_entropy"], s["s2"]["token_logp"],
                                     s["tok_off"], tc, ts)
        asm = ssd.ssd_assemble(s["ids"], s["tok_off"], s["gate"]["gate_accept"],
                               s["s2"]["accepted_len"], s["s2"]["all_accepted"])
        gr = ssd.ssd_greedy_step(s["vb"].logits[:R])
        prep.append((sw, asm, gr))
    torch.cuda.synchronize()

    def timed(fn, n=60):
        for i in range(6):
            fn(i % n_sets)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for i in range(n):
            fn(i % n_sets)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n * 1e3

    t_sw = timed(lambda i: ssd.ssd_threshold_sweep(
        sets[i]["s1"]["utt_max_entropy"], sets[i]["s2"]["token_logp"], sets[i]["tok_off"], tc, ts,
        out=prep[i][0]))
    t_asm = timed(lambda i: ssd.ssd_assemble(
        sets[i]["ids"], sets[i]["tok_off"], sets[i]["gate"]["gate_accept"],
        sets[i]["s2"]["accepted_len"], sets[i]["s2"]["all_accepted"], out=prep[i][1]))
    t_gr = timed(lambda i: ssd.ssd_greedy_step(sets[i]["vb"].logits[:R], out=prep[i][2]))
    # the streaming kernel alone, from events the library records around it
    kev = make_events(2 * KERNEL_LAUNCHES)
    for j in range(KERNEL_LAUNCHES):
        o = ssd.LaunchOpts()
        o.ev_begin, o.ev_end = kev[2 * j].cuda_event, kev[2 * j + 1].cuda_event
        ssd.ssd_greedy_step(sets[j % n_sets]["vb"].logits[:R], out=prep[j % n_sets][2], opts=o)
    torch.cuda.synchronize()
    t_gk = statistics.mean(kev[2 * j].elapsed_time(kev[2 * j + 1]) for j in range(2, KERNEL_LAUNCHES)) * 1e3
    w = sets[0]["w"]
    gbytes = R * w.V_llm * elem_size(w)
    # the whole step with ssd_verify_early_exit in place of ssd_verify (same decisions; the
    # per-token log-likelihoods only up to a little past each first reject)
    code = ssd.BF16 if w.dtype == "bf16" else ssd.F32
    ee = []
    for s in sets:
        o = ssd.alloc_early_exit_outputs(s["M"], s["B"], s["w"].V_llm, code, device)
        ee.append((ssd.bind_verify_early_exit(s["vb"].logits, s["tok_off"], s["ids"],
                                              s["w"].tau_slm, o, skip=s["gate"]["gate_accept"]), o))

    def ee_step(i):
        sets[i]["call_ctc"]()
        sets[i]["call_gate"]()
        ee[i][0]()

    n_ee = max(20, min(400, int(0.05 / max(1e-6, sum(s["verify_bytes"] for s in sets) / n_sets / 5e12))))
    t_ee = timed(ee_step, n_ee)
    same = all(torch.equal(ee[i][1]["accepted_len"], sets[i]["s2"]["accepted_len"]) and
               torch.equal(ee[i][1]["all_accepted"], sets[i]["s2"]["all_accepted"])
               for i in range(n_sets))
    rows_read = sum(int(ee[i][1]["rows_read"].clamp(min=0).sum().item()) for i in range(n_sets))
    fell_back = any(bool((ee[i][1]["rows_read"] < 0).any().item()) for i in range(n_sets))
    rows_full = sum(s["m_active"] for s in sets)
    units = sum(s["B"] for s in sets) / n_sets
    early = {"utterances_per_s": round(units / (t_ee * 1e-6), 1), "us_per_step": round(t_ee, 2),
             "verify_rows_read_frac": None if fell_back else round(rows_read / max(rows_full, 1), 4),
             "same_decisions_as_full": bool(same),
             "note": "separate mode, not part of `value`: rows after an utterance's first reject "
                     "are not read (Section 2.3 needs only the first reject)"}
    del ee
    # one rank's share of a vocabulary-parallel head: a quarter of the columns, then the
    # combination of four ranks' statistics (this GPU's own four slices stand in for them; the
    # all-gather between ranks, 12 bytes per row, needs more than one GPU and is not timed)
    vp = None
    if w.V_llm % 4 == 0:
        vq = w.V_llm // 4
        vsh = []
        for s in sets:
            ws = torch.empty((max(256, ssd.ssd_verify_workspace_bytes(s["B"], s["M"], vq, code)),),
                             dtype=torch.uint8, device=device)
            st = torch.zeros((4, s["M"], 3), dtype=torch.float32, device=device)
            for r in range(4):
                ssd.ssd_verify_shard(s["vb"].logits[:, r * vq:(r + 1) * vq], r * vq, s["tok_off"],
                                     s["ids"], skip=s["gate"]["gate_accept"], stats=st[r],
                                     workspace=ws)
            o = ssd.alloc_verify_outputs(s["M"], s["B"], device, 0)
            ssd.ssd_verify_combine(st, w.V_llm, s["tok_off"], s["ids"], w.tau_slm,
                                   skip=s["gate"]["gate_accept"], out=o)
            vsh.append((ws, st, o))
        torch.cuda.synchronize()
        same_vp = all(torch.equal(vsh[i][2]["accepted_len"], sets[i]["s2"]["accepted_len"])
                      for i in range(n_sets))
        t_sh = timed(lambda i: ssd.ssd_verify_shard(
            sets[i]["vb"].logits[:, vq:2 * vq], vq, sets[i]["tok_off"], sets[i]["ids"],
            skip=sets[i]["gate"]["gate_accept"], stats=vsh[i][1][1], workspace=vsh[i][0]), n_ee)
        t_cb = timed(lambda i: ssd.ssd_verify_combine(
            vsh[i][1], w.V_llm, sets[i]["tok_off"], sets[i]["ids"], w.tau_slm,
            skip=sets[i]["gate"]["gate_accept"], out=vsh[i][2]))
        sh_bytes = rows_full / n_sets * vq * elem_size(w)
        vp = {"ranks": 4, "shard_us": round(t_sh, 2), "combine_us": round(t_cb, 2),
              "shard_gbs": round(sh_bytes / (t_sh * 1e-6) / 1e9, 1),
              "same_decisions_as_full": bool(same_vp),
              "note": "ssd_verify_shard on columns [V/4, V/2) (host-paced call: streaming kernel "
                      "plus its closing kernel) and ssd_verify_combine over four slices' "
                      "statistics; the all-gather between ranks is not part of it"}
        del vsh
    return {"early_exit_step": early, "vocab_parallel_verify": vp,
            "threshold_sweep": {"pairs": len(pairs), "us_per_call": round(t_sw, 2)},
            "assemble": {"us_per_call": round(t_asm, 2),
                         "ar_count": int(prep[0][1]["ar_count"].cpu()[0])},
            "greedy_step": {"rows": R, "V": w.V_llm, "us_per_call": round(t_gr, 2),
                            "kernel_us": round(t_gk, 2),
                            "kernel_gbs": round(gbytes / (t_gk * 1e-6) / 1e9, 1),
                            "kernel_frac": round(gbytes / (t_gk * 1e-6) / 1e9 / peak, 4),
                            "note": "us_per_call is host-paced (Python marshalling included); "
                                    "kernel_* is the streaming kernel between two events; rows "
                                    "from %d input sets in turn" % n_sets}}


def run_e2e(s, device, steps, D, world):
    """The same path through the public binding with every input starting in pinned host
    memory: each step copies the logits, offsets and draft ids to the device, makes the three
    calls and reads the per-utterance decisions and the draft back to the host."""
    import torch
    w = s["w"]

    def pin(t):
        h = torch.empty(t.shape, dtype=t.dtype, pin_memory=True)
        h.copy_(t)
        return h
    h_in = dict(ctc=pin(s["cb"].logits), llm=pin(s["vb"].logits), off=pin(s["off"]),
                tok_off=pin(s["tok_off"]), ids=pin(s["ids"]))
    d_in = dict(ctc=s["cb"].logits, llm=s["vb"].logits, off=s["off"], tok_off=s["tok_off"],
                ids=s["ids"])
    outs = [s["s1"]["draft_tokens"], s["s1"]["draft_len"], s["s1"]["utt_max_entropy"],
            s["gate"]["gate_accept"], s["s2"]["accepted_len"], s["s2"]["all_accepted"],
            s["s2"]["token_logp"], s["s1"]["utt_status"], s["s2"]["utt_status"]]
    h_out = [torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in outs]
    h2d = sum(t.numel() * t.element_size() for t in h_in.values())
    d2h = sum(t.numel() * t.element_size() for t in outs)

    def one():
        for k in h_in:
            d_in[k].copy_(h_in[k], non_blocking=True)
        step(s)
        for d, h in zip(outs, h_out):
            h.copy_(d, non_blocking=True)
        torch.cuda.current_stream().synchronize()      # the caller reads the decisions now

    for _ in range(1 if h2d > 2e9 else 3):
        one()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    D.barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    e0.record()
    for _ in range(steps):
        one()
    e1.record()
    torch.cuda.synchronize()
    wall = time.perf_counter() - t0
    D.barrier()
    # host waits are part of this number: take the larger of device and wall time
    sec = max(e0.elapsed_time(e1) * 1e-3, wall)
    sec_max, units = D.reduce_max_sum(sec, float(steps * s["B"]), device)
    del h_in
    return {"value": round(units / sec_max, 1), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
            "d2h_bytes_per_step": int(d2h), "steps": steps,
            "ms_per_step": round(sec_max / steps * 1e3, 4),
            "h2d_gbs": round(h2d * steps / sec_max / 1e9, 1),
            "note": "pinned host -> device copies of all logits, three C-ABI calls, decisions "
                    "and draft copied back, stream synchronised every step"}


# ---- the oracle as a CPU baseline ------------------------------------------------------------
def host_inputs(s, n_utt):
    """Host copies (in the form the oracle takes) of the first n_utt utterances of a batch."""
    import numpy as np
    import torch

    def to_np(t):
        t = t.detach().cpu().contiguous()
        if t.dtype == torch.bfloat16:
            return t.view(torch.int16).numpy().view(np.uint16)
        return t.numpy()
    off, tok = s["cb"].frame_off.numpy(), s["vb"].tok_off.numpy()
    f1, k1 = int(off[n_utt]), int(tok[n_utt])
    return dict(ctc=to_np(s["cb"].logits[:f1]), llm=to_np(s["vb"].logits[:k1]),
                off=off[:n_utt + 1], tok_off=tok[:n_utt + 1], ids=s["vb"].draft_ids.numpy()[:k1])


def oracle_pass(h, w, lo, hi):
    """The oracle's whole path on utterances [lo, hi) of a host batch; returns seconds."""
    import numpy as np
    from oracle import ref
    off, tok = h["off"], h["tok_off"]
    f0, f1, k0, k1 = int(off[lo]), int(off[hi]), int(tok[lo]), int(tok[hi])
    t0 = time.perf_counter()
    o1 = ref.ctc_draft(h["ctc"][f0:f1], w.V_ctc, off[lo:hi + 1] - f0, w.blank_id, w.max_draft_len)
    g = ref.entropy_gate(o1["frame_entropy"], off[lo:hi + 1] - f0, float(np.float32(w.tau_ctc)))
    ref.verify(h["llm"][k0:k1], w.V_llm, tok[lo:hi + 1] - k0, h["ids"][k0:k1],
               float(np.float32(w.tau_slm)), skip=g["gate_accept"])
    return time.perf_counter() - t0


def cpu_baseline(s, budget_s, single_thread_too=False):
    """The oracle as it stands on the host cores, one utterance per thread, on a bounded sample:
    the first utterances of the batch, as many as about `budget_s` seconds of wall time allow
    (at least one per thread).  With single_thread_too, one thread on a few utterances as well."""
    from oracle import ref
    w = s["w"]
    cores = len(os.sched_getaffinity(0))
    threads = ref.set_threads(max(1, min(cores, w.B)))
    first = min(w.B, threads)
    h = host_inputs(s, first)
    t1 = oracle_pass(h, w, 0, first)            # one utterance per thread
    n = int(min(w.B, max(first, first * budget_s / max(t1, 1e-9))))
    n -= n % threads if n > threads else 0
    if n > first:
        h = host_inputs(s, n)
    reps = int(max(1, min(50, round(budget_s / max(t1 * n / first, 1e-9)))))
    sec = sum(oracle_pass(h, w, 0, n) for _ in range(reps))
    rec = {"value": round(n * reps / sec, 2), "unit": UNIT, "cores": threads, "kind": "oracle",
           "sample": "first %d of the %d utterances of one batch, whole path (fp64 two-pass C "
                     "oracle, one utterance per thread), %d pass(es), %.1f s wall = %.0f "
                     "core-seconds" % (n, w.B, reps, sec, sec * threads)}
    if single_thread_too:
        ref.set_threads(1)
        m = max(1, min(n, int(round(0.25 * budget_s / max(t1, 1e-9)))))   # t1 ~ one utterance on one core
        sec1 = oracle_pass(h, w, 0, m)
        ref.set_threads(threads)
        rec["single_thread"] = {"value": round(m / sec1, 2), "unit": UNIT, "cores": 1,
                                "sample": "first %d utterance(s), %.1f s" % (m, sec1)}
    return rec


def run_reference(args):
    """Times the CPU oracle on this arm's workload; rank 0 only."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    import torch
    from oracle import ref
    from paper_2603_11243_b200 import synth
    base = synth.CONFIGS[args.config]
    K, W = args.steps, args.warmup
    cores = len(os.sched_getaffinity(0))
    threads = ref.set_threads(max(1, min(cores, base.B)))
    # The oracle sees a bounded sample of the workload: a smaller batch of the same configuration
    # (same generators and value mix, fewer utterances), since it could not get through the full
    # batch of the larger configurations in minutes.
    pool = int(min(base.B, 2 * threads))
    w = synth.scaled(base, B=pool)

    def to_np(t):
        t = t.contiguous()
        return t.view(torch.int16).numpy().view(np.uint16) if t.dtype == torch.bfloat16 else t.numpy()
    cb = synth.make_ctc_batch(w, "cpu")
    ctc = to_np(cb.logits)
    # the oracle's own drafts size the verify batch, as the GPU arm's drafts size its batch
    o1 = ref.ctc_draft(ctc, w.V_ctc, cb.frame_off.numpy(), w.blank_id, w.max_draft_len)
    vb = synth.make_verify_batch(w, o1["draft_len"].tolist(), "cpu")
    h = dict(ctc=ctc, llm=to_np(vb.logits), off=cb.frame_off.numpy(), tok_off=vb.tok_off.numpy(),
             ids=vb.draft_ids.numpy())
    # bounded sample per step: u utterances, sized so that K + W steps take about two minutes
    probe = oracle_pass(h, w, 0, min(pool, threads)) / min(pool, threads)
    u = int(max(1, min(pool, 100.0 / max(K + W, 1) / max(probe, 1e-9))))
    starts = [(i * u) % max(1, pool - u + 1) for i in range(K + W)]
    for i in range(W):
        oracle_pass(h, w, starts[i], starts[i] + u)
    t0 = time.perf_counter()
    for i in range(W, W + K):
        oracle_pass(h, w, starts[i], starts[i] + u)
    sec = time.perf_counter() - t0
    value = K * u / sec
    sample = ("%d utterance(s) per step out of a %d-utterance batch of configs[%d] (window "
              "sliding over them), whole path in the fp64 C oracle, %d thread(s)" %
              (u, pool, args.config, threads))
    line = {"impl": "reference", "metric": METRIC, "value": round(value, 3), "unit": UNIT,
            "n_gpus": args.gpus, "steps": K, "warmup": W, "ms_per_step": round(sec / K * 1e3, 3),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic",
            "config": {"workload": "configs[%d] %s (CPU oracle on a bounded sample per step)" %
                                   (args.config, base.name), "sample": sample},
            "cpu_baseline": {"value": round(value, 3), "unit": UNIT, "cores": threads,
                             "kind": "oracle", "sample": sample},
            "e2e": {"value": round(value, 3), "unit": UNIT, "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---- the throughput sweep ------------------------------------------------------------------
SWEEP_B = (1, 8, 64, 256, 1024)
SWEEP_V = (32000, 49152, 100352, 152064)
SWEEP_DTYPES = ("f32", "bf16")
SWEEP_MAX_RESIDENT = 48e9        # bytes of logits generated at a time; larger points run as
                                 # equal sub-batches, each timed on its own, times added


def run_sweep(args):
    import torch
    from paper_2603_11243_b200 import build as lib_build
    from paper_2603_11243_b200 import synth
    lib_build.build()
    device = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    peak, peak_kind = peaks()
    with open(args.sweep, "a") as out:
        for dtype in SWEEP_DTYPES:
            for V in SWEEP_V:
                for B in SWEEP_B:
                    w = synth.sweep_point(B, V, dtype)
                    if args.sweep_filter and args.sweep_filter not in w.name:
                        continue
                    es = elem_size(w)
                    est = B * (1000 * w.V_ctc + 250 * V) * es
                    n_sub = max(1, math.ceil(est / SWEEP_MAX_RESIDENT))
                    while B % n_sub:
                        n_sub += 1
                    n_sets = max(1, min(8, math.ceil(4e8 / (est / n_sub))))
                    steps = int(max(10, min(300, 0.25 / (est / n_sub / 5e12))))
                    ms = t_ctc = t_ver = 0.0
                    ctc_b = ver_b = 0
                    launches = 0.0
                    for sub in range(n_sub):
                        ws = synth.scaled(w, B=B // n_sub, seed=w.seed + 31 * sub)
                        sets = build_sets(ws, device, n_sets)
                        a, _, nl = timed_steps(sets, steps, 5)
                        b, c, cb_, vb_ = time_kernels(sets)
                        ms, t_ctc, t_ver = ms + a / steps, t_ctc + statistics.mean(b), t_ver + statistics.mean(c)
                        launches += nl / steps
                        ctc_b += cb_
                        ver_b += vb_
                        del sets
                        torch.cuda.empty_cache()
                    nbytes = ctc_b + ver_b
                    line = {"point": w.name, "B": B, "V_llm": V, "dtype": dtype,
                            "sub_batches": n_sub, "input_sets": n_sets, "steps": steps,
                            "logits_bytes": int(nbytes), "ms_per_step": round(ms, 5),
                            "gpu_launches_per_step": launches,
                            "utterances_per_s": round(B / (ms * 1e-3), 1),
                            "step_gbs": round(nbytes / (ms * 1e-3) / 1e9, 1),
                            "step_frac": round(nbytes / (ms * 1e-3) / 1e9 / peak, 4),
                            "ctc_us": round(t_ctc * 1e3, 2),
                            "ctc_gbs": round(ctc_b / (t_ctc * 1e-3) / 1e9, 1),
                            "ctc_frac": round(ctc_b / (t_ctc * 1e-3) / 1e9 / peak, 4),
                            "verify_us": round(t_ver * 1e3, 2),
                            "verify_gbs": round(ver_b / (t_ver * 1e-3) / 1e9, 1) if t_ver else None,
                            "verify_frac": round(ver_b / (t_ver * 1e-3) / 1e9 / peak, 4) if t_ver else None,
                            "peak_gbs": peak, "peak_kind": peak_kind}
                    out.write(json.dumps(line) + "\n")
                    out.flush()
                    print(json.dumps(line), flush=True)


def run_stage1_only(args):
    """Stage 1 alone on one configuration's CTC batch, for a profiler capture of its kernels."""
    import torch
    from paper_2603_11243_b200 import binding as ssd
    from paper_2603_11243_b200 import build as lib_build
    from paper_2603_11243_b200 import synth
    lib_build.build()
    device = torch.device("cuda", 0)
    w = synth.CONFIGS[args.config]
    cb = synth.make_ctc_batch(w, device)
    off = cb.frame_off.to(device)
    out = ssd.alloc_ctc_outputs(cb.logits.shape[0], w.B, device)
    for _ in range(3):
        ssd.ssd_ctc_draft(cb.logits, off, w.blank_id, w.max_draft_len, out=out)
    torch.cuda.synchronize()
    print(json.dumps({"stage1_only": w.name, "frames": int(cb.logits.shape[0]), "V_ctc": w.V_ctc,
                      "dtype": w.dtype, "calls": 3}))


def run_verify_rows_only(args):
    """ssd_verify alone on a few thousand rows of one configuration's LLM vocabulary (a GB or
    two on the device), for a profiler capture of its kernels."""
    import torch
    from paper_2603_11243_b200 import binding as ssd
    from paper_2603_11243_b200 import build as lib_build
    from paper_2603_11243_b200 import synth
    lib_build.build()
    device = torch.device("cuda", 0)
    base = synth.CONFIGS[args.config]
    per = min(base.max_draft_len, 200)
    B = max(1, args.ncu_rows // per)
    w = synth.scaled(base, B=B)
    vb = synth.make_verify_batch(w, [per] * B, device)
    for _ in range(3):
        ssd.ssd_verify(vb.logits, vb.tok_off.to(device), vb.draft_ids.to(device), w.tau_slm)
    torch.cuda.synchronize()
    print(json.dumps({"verify_only": w.name, "rows": int(vb.logits.shape[0]), "V_llm": w.V_llm,
                      "dtype": w.dtype, "calls": 3}))


def main():
    args = parse_args()
    if args.sweep:
        run_sweep(args)
        return
    if args.ncu_stage1:
        run_stage1_only(args)
        return
    if args.ncu_rows:
        run_verify_rows_only(args)
        return
    if args.impl == "reference":
        run_reference(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1",
               "--nproc-per-node", str(args.gpus), "--master-addr", "127.0.0.1",
               "--master-port", "29533", os.path.abspath(__file__)] + sys.argv[1:]
        raise SystemExit(subprocess.call(cmd))
    run_ours(args)


if __name__ == "__main__":
    main()
