#!/usr/bin/env python
"""Benchmark of the prefix-shared DPO hot path on B200.

One "step" is one pass of the whole path over one synthetic pack: psa_plan on the
host, psa_fwd, psa_bwd, and dpo_logp over the pack's logits.  The headline metric
is the useful TFLOP/s of attention forward + backward (14*d*Hq*U flops, U = the
unmasked (q, kv) pairs per head) over the time of those two calls, measured with
CUDA events inside the timed steps; packed tokens/s over the whole step and the
gather's GB/s are reported beside it.  The default workload is the largest
single-GPU configuration (multi-turn, a 32768-token pack, with the gather over bf16
logits of vocabulary 128256); the other three configurations are measured in the
same process and reported in the line's `workloads` object.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 1..4] [--impl reference]

N > 1 (launched through torch.distributed.run) shards the batch by packs: every rank
takes a pack of its own (the packs of a batch are independent), so there is no
collective on the data path; the report sums the ranks' work over the slowest time.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "psa_attention_fwd_bwd_useful_tflops"
UNIT = "TFLOP/s"
VOCAB = 128256            # logits width of the gather leg (bf16)
NOMINAL_BF16_TFLOPS = 2250.0
NOMINAL_HBM_GBS = 8000.0
TARGET_FRAC_OF_BF16_PEAK = 0.5      # attention fwd+bwd, useful flops
TARGET_FRAC_OF_HBM = 0.7            # the gather
MIN_TIMED_SECONDS = 0.5             # the timed region runs at least this long (inner repeats of the step)
N_E2E = int(os.environ.get("PSA_BENCH_E2E_STREAMS", "3"))   # arenas / streams of the end-to-end leg
ORACLE_SAMPLE_PAIRS = 6.0e6         # useful pairs per head of the oracle's timed sample (about 1.5 s per pass)
NCU_TRAFFIC_FILE = os.path.join(ROOT, "profiles", "ncu_traffic.json")
# sources whose text decides the DRAM traffic of the backward's main kernel (kernel, waits, launch order)
TRAFFIC_SOURCES = ("psa_bwd.cu", "psa_device.cuh", "psa_plan.cpp")


def measured_peaks():
    """Roofline denominators: the measured copy bandwidth and cuBLAS bf16 rate of
    this machine's B200s if the driver left them, else an earlier measurement."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def traffic_source_digest():
    """Digest of the sources that decide the backward kernel's DRAM traffic; an ncu figure taken
    from another version of them is stale."""
    h = hashlib.sha256()
    for name in TRAFFIC_SOURCES:
        with open(os.path.join(ROOT, "paper_2410_20305_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def ncu_traffic(kernel, workload_name):
    """DRAM bytes (read + write) of one launch of `kernel` on `workload_name`, from the tracked
    summary of an ncu capture (written by paper_2410_20305_b200/ncu_summary.py); None when there
    is no capture of this workload or it was taken from other kernel sources."""
    try:
        rec = json.load(open(NCU_TRAFFIC_FILE))[kernel][workload_name]
    except (OSError, KeyError, ValueError):
        return None, "no capture of this kernel on this workload"
    if rec.get("source_digest") != traffic_source_digest():
        return None, "stale: captured from other kernel sources (%s)" % rec.get("source_digest")
    return float(rec["dram_bytes"]), rec.get("command")


class ClockSampler:
    """Samples the SM clock and the clock-event (throttle) reasons while the timed region runs:
    NVML from a thread of this process every 2 ms (read-only queries); nvidia-smi as a fallback."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
    BITS = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4}

    def __init__(self, index):
        self.index, self.rows, self.proc, self.thread = index, [], None, None
        self.sm, self.max_sm, self.mask, self.stop, self.source = [], None, 0, False, None

    def _nvml_handle(self):
        import pynvml
        pynvml.nvmlInit()
        visible = os.environ.get("CUDA_VISIBLE_DEVICES")
        idx = self.index
        if visible:   # the CUDA ordinal indexes the visible list, NVML the physical one
            ids = [v.strip() for v in visible.split(",") if v.strip()]
            if idx < len(ids):
                if ids[idx].isdigit():
                    idx = int(ids[idx])
                else:
                    return pynvml, pynvml.nvmlDeviceGetHandleByUUID(ids[idx])
        return pynvml, pynvml.nvmlDeviceGetHandleByIndex(idx)

    def _poll(self, pynvml, h):
        reasons = getattr(pynvml, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
            pynvml.nvmlDeviceGetCurrentClocksThrottleReasons
        while not self.stop:
            try:
                self.sm.append(float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)))
                self.mask |= int(reasons(h))
            except Exception:
                break
            time.sleep(0.002)

    def __enter__(self):
        try:
            pynvml, h = self._nvml_handle()
            self.max_sm = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            self.source = "nvml"
            self.thread = threading.Thread(target=self._poll, args=(pynvml, h), daemon=True)
            self.thread.start()
            return self
        except Exception:
            self.source = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.source = "nvidia-smi"
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def __exit__(self, *a):
        self.stop = True
        if self.proc:
            self.proc.terminate()
            self.proc.wait()
        if self.thread:
            self.thread.join(timeout=2)

    def summary(self):
        if self.source == "nvml":
            reasons = [n for n in self.NAMES if self.mask & self.BITS[n]]
            return {"sm_mhz": float(np.median(self.sm)) if self.sm else None, "sm_min_mhz": min(self.sm) if self.sm else None,
                    "sm_max_mhz": self.max_sm, "reasons": reasons, "samples": len(self.sm), "source": "nvml, every 2 ms"}
        sm = [float(r[0]) for r in self.rows if len(r) >= 6 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 6 and r[1].replace(".", "").isdigit()]
        reasons = [n for i, n in enumerate(self.NAMES) if any(len(r) >= 6 and r[2 + i] == "Active" for r in self.rows)]
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm), "source": "nvidia-smi -lms 20"}


def max_over_ranks(values, device):
    """Element-wise maximum of a list of floats over all ranks (identity on one rank).
    The path has no exchange step: this reduction of the timings is the only collective."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def sum_over_ranks(values, device):
    """Element-wise sum of a list of floats over all ranks (identity on one rank): the work the
    ranks did on their own packs.  Like max_over_ranks it reduces a few scalars of the report,
    after the timed region; the data path has no collective."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return [float(x) for x in t.cpu()]


def whole_job_tflops(flops_all_ranks, ms):
    """The packs of a batch are independent: every rank takes its own pack; the job's work is the
    sum over the ranks, its time the slowest rank's."""
    return flops_all_ranks / ms / 1e9


def rank_pack(workload, rank):
    """Rank 0 takes the configuration's own pack; every other rank draws another pack of the same
    length distribution (pack sharding: one pack of the batch per GPU)."""
    from paper_2410_20305_b200 import workloads as wl
    return wl.config_pack(workload) if rank == 0 else wl.config_pack(workload, seed=1000 + workload + 7919 * rank)


def oracle_sample_set(pack):
    """The bounded sample of the workload that both oracle legs time: whole samples of the pack
    (attention is independent per sample, which the oracle's own tests pin), taken at every second
    rank of the samples sorted by length so that the length mix is the pack's, until their useful
    pairs reach ORACLE_SAMPLE_PAIRS; one kv-head group (4 query heads, 1 kv head)."""
    from oracle import psa_oracle as orc
    order = np.argsort(pack.cu_seqlens[1:] - pack.cu_seqlens[:-1], kind="stable")
    chosen, pairs = [], 0
    for s in [int(x) for x in order[0::2]]:
        chosen.append(s)
        pairs += orc.useful_pairs([pack.prefix_len[s]], [pack.chosen_len[s]], [pack.rejected_len[s]])
        if pairs >= ORACLE_SAMPLE_PAIRS:
            break
    return chosen


def oracle_sample(pack, steps, warmup):
    """Times the fp64 oracle, as it stands, on oracle_sample_set(pack): forward and backward, dense
    mask, numpy.  Returns (useful TFLOP/s, description, cores, seconds per step)."""
    import torch
    from oracle import psa_oracle as orc
    from paper_2410_20305_b200 import workloads as wl
    chosen = oracle_sample_set(pack)
    subs, flops = [], 0.0
    for s in chosen:
        P, C, R = int(pack.prefix_len[s]), int(pack.chosen_len[s]), int(pack.rejected_len[s])
        sub = wl.pack_from_lengths("sample", [(P, C, R)], 4, 1, pack.head_dim)
        q, k, v, d_o = (wl.to_f64(t) for t in wl.attention_inputs(sub, 2000 + s, std=1.0))
        mask = orc.packed_mask(sub.cu_seqlens, sub.prefix_len, sub.chosen_len, sub.rejected_len)
        subs.append((q, k, v, d_o, mask))
        flops += 14.0 * pack.head_dim * 4 * orc.useful_pairs([P], [C], [R])
    times = []
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        for q, k, v, d_o, mask in subs:
            orc.attention_fwd(q, k, v, mask)
            orc.attention_bwd(q, k, v, d_o, mask)
        if i >= warmup:
            times.append(time.perf_counter() - t0)
    sec = float(np.mean(times))
    desc = "%d of the pack's %d samples (%d of %d tokens, every second one by length), 4 query heads / 1 kv head, " \
           "fwd+bwd, dense fp64 numpy" % (len(chosen), pack.n_samples,
                                          int(sum(pack.cu_seqlens[s + 1] - pack.cu_seqlens[s] for s in chosen)),
                                          pack.total_tokens)
    return flops / sec / 1e12, desc, torch.get_num_threads(), sec


def run_reference(args, pack, rank):
    """The reference arm: the CPU oracle on the machine's host cores, rank 0 only, on the same sample
    as the cpu_baseline leg of the main arm."""
    if rank != 0:
        return
    val, desc, cores, sec = oracle_sample(pack, args.steps, args.warmup)
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": pack.name, "sample": desc},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def attention_record(index, dev, peaks, iters=30, warm=5):
    """Attention fwd+bwd of workload `index` on the shared layout and, with the same kernels, on the
    unshared paired layout: ms, useful TFLOP/s, fractions of the bf16 peaks, tokens/s, speed-up."""
    import torch
    from paper_2410_20305_b200 import binding as B
    from paper_2410_20305_b200 import workloads as wl
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def timed(pk, seed):
        Hq, Hkv, d = pk.n_q_heads, pk.n_kv_heads, pk.head_dim
        q, k, v, d_o = (t.to(dev) for t in wl.attention_inputs(pk, seed))
        plan = B.psa_plan(pk.cu_seqlens, pk.prefix_len, pk.chosen_len, pk.rejected_len, Hq, Hkv, d)
        o, lse = B.psa_fwd(plan, q, k, v)
        ws = torch.empty(plan.bwd_workspace_bytes, dtype=torch.uint8, device=dev)
        dq, dk, dv = B.psa_bwd(plan, d_o, q, k, v, o, lse, workspace=ws)
        for _ in range(warm):
            B.psa_fwd(plan, q, k, v, o=o, lse=lse)
            B.psa_bwd(plan, d_o, q, k, v, o, lse, dq=dq, dk=dk, dv=dv, workspace=ws)
        torch.cuda.synchronize()
        a, m, b = ev(), ev(), ev()
        fwd_ms = 0.0
        a.record()
        for _ in range(iters):
            B.psa_fwd(plan, q, k, v, o=o, lse=lse)
            B.psa_bwd(plan, d_o, q, k, v, o, lse, dq=dq, dk=dk, dv=dv, workspace=ws)
        b.record()
        torch.cuda.synchronize()
        total = a.elapsed_time(b) / iters
        a.record()
        for _ in range(iters):
            B.psa_fwd(plan, q, k, v, o=o, lse=lse)
        m.record()
        torch.cuda.synchronize()
        fwd_ms = a.elapsed_time(m) / iters
        return total, fwd_ms, plan.useful_pairs, plan.live_tiles

    pack = wl.config_pack(index)
    Hq, Hkv, d, T = pack.n_q_heads, pack.n_kv_heads, pack.head_dim, pack.total_tokens
    ms, fwd_ms, U, live = timed(pack, 2000 + index)
    pp = pack.paired()
    p_ms, _, pU, _ = timed(pp, 2100 + index)
    torch.cuda.empty_cache()
    tflops = 14.0 * d * Hq * U / ms / 1e9
    min_bytes = T * (6 * Hq + 6 * Hkv) * d * 2
    return {"workload": pack.name, "total_tokens": T, "n_samples": pack.n_samples, "useful_pairs_per_head": U,
            "live_tiles": live, "attention_fwd_bwd_ms": ms, "fwd_ms_back_to_back": fwd_ms, "useful_tflops": tflops,
            "pct_of_bf16_peak": {"measured": tflops / peaks["bf16_tflops"], "nominal": tflops / NOMINAL_BF16_TFLOPS},
            "attention_tokens_per_s": T / (ms * 1e-3),
            "attention_min_hbm_frac": {"measured": min_bytes / ms / 1e6 / peaks["hbm_gbs"],
                                       "nominal": min_bytes / ms / 1e6 / NOMINAL_HBM_GBS},
            "paired_layout": {"tokens": pp.total_tokens, "fwd_bwd_ms": p_ms, "speedup_shared_over_paired": p_ms / ms,
                              "ideal_pair_ratio": pU / U, "token_ratio": pp.total_tokens / T},
            "timing": "%d iterations after %d warm-up, CUDA events, inputs larger than L2" % (iters, warm)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="psa", choices=["psa", "reference"])
    ap.add_argument("--workload", type=int, default=3, choices=[1, 2, 3, 4],
                    help="1 llama3-8b, 2 long-prompt, 3 multi-turn (default: the largest single-GPU configuration), 4 short-many")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-layer", action="store_true")
    ap.add_argument("--no-paired", action="store_true")
    ap.add_argument("--no-workloads", action="store_true", help="skip the records of the other three configurations")
    ap.add_argument("--no-logp", action="store_true", help="attention only (small footprint, for ncu captures)")
    ap.add_argument("--no-inner-repeats", action="store_true", help="time exactly --steps passes (for ncu captures)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    from paper_2410_20305_b200 import workloads as wl
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    pack = rank_pack(args.workload, rank)
    if args.impl == "reference":
        return run_reference(args, pack, rank)

    import torch
    import torch.distributed as dist
    import paper_2410_20305_b200 as psa
    from paper_2410_20305_b200 import binding as B
    from paper_2410_20305_b200.layer import AttentionLayer

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    peaks = measured_peaks()

    T, Hq, Hkv, d = pack.total_tokens, pack.n_q_heads, pack.n_kv_heads, pack.head_dim
    q, k, v, d_o = (t.to(dev) for t in wl.attention_inputs(pack, 2000 + args.workload, std=1.0))
    gen = torch.Generator(device=dev).manual_seed(3000 + args.workload + rank)
    n_logit_rows = 8 if args.no_logp else T
    logits = torch.empty((n_logit_rows, VOCAB), dtype=torch.bfloat16, device=dev)
    for lo in range(0, n_logit_rows, 2048):   # N(0, variance 3), generated in slabs to bound the fp32 temporary
        hi = min(n_logit_rows, lo + 2048)
        logits[lo:hi] = (torch.randn((hi - lo, VOCAB), generator=gen, device=dev) * 3.0 ** 0.5).to(torch.bfloat16)
    tok = torch.randint(0, VOCAB, (T,), generator=gen, device=dev, dtype=torch.int32).cpu().numpy()
    targets, seg, fr, ft, fs = psa.logp_labels(tok, pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    i32 = lambda a: torch.as_tensor(np.asarray(a, dtype=np.int32)).to(dev)
    targets, seg_d, fr, ft, fs = i32(targets), i32(seg), i32(fr), i32(ft), i32(fs)
    n_seg = 2 * pack.n_samples
    live_rows = int((seg >= 0).sum()) + int(((seg < 0)[fr.cpu().numpy()]).sum() if len(fr) else 0)

    plan0 = B.psa_plan(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len, Hq, Hkv, d)
    o = torch.empty_like(q); lse = torch.empty((Hq, T), dtype=torch.float32, device=dev)
    dq = torch.empty_like(q); dk = torch.empty_like(k); dv = torch.empty_like(v)
    ws = torch.empty(plan0.bwd_workspace_bytes, dtype=torch.uint8, device=dev)
    logp = torch.empty(n_seg, dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    U = plan0.useful_pairs
    flops_fwd, flops_bwd = 4.0 * d * Hq * U, 10.0 * d * Hq * U

    ev = lambda: torch.cuda.Event(enable_timing=True)
    KERNELS = (("fwd", 0), ("bwd", 1), ("logp", 2), ("bwd_delta_clear", 3), ("bwd_convert", 4))

    def step(e0=None, e1=None, e2=None, kev=None):
        # kev: this pass's own event pairs, which the library records right around each kernel
        if kev is not None:
            for (name, which), pair in zip(KERNELS, kev):
                B.psa_profile_events(which, pair[0], pair[1], created=True)
        plan = B.psa_plan(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len, Hq, Hkv, d)
        if e0 is not None:
            e0.record()
        B.psa_fwd(plan, q, k, v, o=o, lse=lse, status=status)
        B.psa_bwd(plan, d_o, q, k, v, o, lse, dq=dq, dk=dk, dv=dv, workspace=ws, status=status)
        if e1 is not None:
            e1.record()
        if not args.no_logp:
            B.dpo_logp(logits, targets, seg_d, n_seg, fr, ft, fs, out=logp, status=status)
        if e2 is not None:
            e2.record()
        return plan

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # Planning cost on the host (build + enqueue the upload + destroy), outside the timed region.
    t0 = time.perf_counter()
    for _ in range(20):
        B.psa_plan(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len, Hq, Hkv, d).close()
    plan_host_ms = (time.perf_counter() - t0) * 1e3 / 20

    # Warm-up; the last warm-up steps also give the step's duration, from which the number of inner
    # repeats follows: the timed region is to last at least MIN_TIMED_SECONDS whatever --steps is.
    for i in range(args.warmup):
        step()
    sync_all()
    a, b = ev(), ev()
    a.record()
    for _ in range(3):
        step()
    b.record()
    sync_all()
    est_ms = a.elapsed_time(b) / 3
    inner = 1 if args.no_inner_repeats else max(1, int(math.ceil(MIN_TIMED_SECONDS * 1e3 / (args.steps * est_ms))))
    n_pass = args.steps * inner

    # Every pass of the timed region has its own events: around the attention calls, after the
    # gather, and (recorded by the library itself) right around each kernel.  They are created, i.e.
    # recorded once, before the region starts; nothing inside the region synchronises.
    e_att0, e_att1, e_lp1 = [ev() for _ in range(n_pass)], [ev() for _ in range(n_pass)], [ev() for _ in range(n_pass)]
    k_ev = [[(ev(), ev()) for _ in KERNELS] for _ in range(n_pass)]
    for pairs in k_ev:
        for a_, b_ in pairs:
            a_.record(); b_.record()
    sync_all()
    t_start, t_stop = ev(), ev()
    with ClockSampler(local_rank) as clocks:
        t_start.record()
        for i in range(n_pass):
            step(e_att0[i], e_att1[i], e_lp1[i], k_ev[i])
        t_stop.record()
        sync_all()
    for _, which in KERNELS:
        B.psa_profile_events(which)
    kernel_ms = {name: float(np.mean([k_ev[i][j][0].elapsed_time(k_ev[i][j][1]) for i in range(n_pass)]))
                 for j, (name, _) in enumerate(KERNELS) if not (name == "logp" and args.no_logp)}
    kernel_ms.setdefault("logp", float("nan"))
    timed_ms = t_start.elapsed_time(t_stop)
    step_ms = timed_ms / n_pass
    att_all = [e_att0[i].elapsed_time(e_att1[i]) for i in range(n_pass)]
    att_ms = float(np.mean(att_all))
    lp_ms = float(np.mean([e_att1[i].elapsed_time(e_lp1[i]) for i in range(n_pass)]))
    if int(status.item()) != 0:
        raise SystemExit("device status word is %d: results invalid" % int(status.item()))

    # ---- next step of the path (outside the timed step): DPO loss and its gradient into the logits
    loss_bwd = None
    if not args.no_logp and rank == 0:
        dlogits = torch.empty_like(logits)
        ref_lp = logp * 0.97
        loss_t, coef = B.dpo_loss(logp, ref_lp, 0.1)
        for _ in range(2):
            B.dpo_logp_bwd(logits, targets, seg_d, coef, fr, ft, fs, dlogits=dlogits, status=status)
        torch.cuda.synchronize()
        a, b = ev(), ev()
        a.record()
        for _ in range(5):
            B.dpo_logp_bwd(logits, targets, seg_d, coef, fr, ft, fs, dlogits=dlogits, status=status)
        b.record()
        torch.cuda.synchronize()
        lb_ms = a.elapsed_time(b) / 5
        lb_bytes = live_rows * VOCAB * 2 * 2 + (T - live_rows) * VOCAB * 2     # live rows read + written, dead rows zeroed
        loss_bwd = {"dpo_loss": float(loss_t.item()), "dpo_logp_bwd_ms": lb_ms, "dpo_logp_bwd_gbs": lb_bytes / lb_ms / 1e6,
                    "algorithmic_bytes": lb_bytes}
        del dlogits

    # ---- the gather with every row scored (a longer stream: T x V x 2 bytes), timed alone
    all_rows = None
    if not args.no_logp and rank == 0:
        seg_all = torch.from_numpy((np.arange(T) % n_seg).astype(np.int32)).to(dev)
        for _ in range(2):
            B.dpo_logp(logits, targets, seg_all, n_seg, out=logp.clone(), status=status)
        torch.cuda.synchronize()
        a, b = ev(), ev()
        scratch = torch.empty_like(logp)
        a.record()
        for _ in range(5):
            B.dpo_logp(logits, targets, seg_all, n_seg, out=scratch, status=status)
        b.record()
        torch.cuda.synchronize()
        ar_ms = a.elapsed_time(b) / 5
        ar_bytes = T * (VOCAB * 2 + 8)
        all_rows = {"rows": T, "ms": ar_ms, "gbs": ar_bytes / ar_ms / 1e6, "algorithmic_bytes": ar_bytes}
    del logits
    torch.cuda.empty_cache()

    # ---- the same kernels on the unshared paired layout (2n causal sequences)
    paired = None
    if not args.no_paired and rank == 0:
        pp = pack.paired()
        pq, pk, pv, pdo = (t.to(dev) for t in wl.attention_inputs(pp, 2100 + args.workload))
        pplan = B.psa_plan(pp.cu_seqlens, pp.prefix_len, pp.chosen_len, pp.rejected_len, Hq, Hkv, d)
        po, plse = B.psa_fwd(pplan, pq, pk, pv)
        pws = torch.empty(pplan.bwd_workspace_bytes, dtype=torch.uint8, device=dev)
        pdq, pdk, pdv = B.psa_bwd(pplan, pdo, pq, pk, pv, po, plse, workspace=pws)
        torch.cuda.synchronize()
        a, b = ev(), ev()
        n_p = max(args.steps, 20)
        a.record()
        for _ in range(n_p):
            B.psa_fwd(pplan, pq, pk, pv, o=po, lse=plse)
            B.psa_bwd(pplan, pdo, pq, pk, pv, po, plse, dq=pdq, dk=pdk, dv=pdv, workspace=pws)
        b.record()
        torch.cuda.synchronize()
        p_ms = a.elapsed_time(b) / n_p
        paired = {"tokens": pp.total_tokens, "fwd_bwd_ms": p_ms, "speedup_shared_over_paired": p_ms / att_ms,
                  "ideal_pair_ratio": pplan.useful_pairs / U, "token_ratio": pp.total_tokens / T}
        del pq, pk, pv, pdo, po, plse, pws, pdq, pdk, pdv
        torch.cuda.empty_cache()

    # ---- the other three configurations, measured here and now with the same build
    others = None
    if not args.no_workloads and rank == 0:
        others = {}
        for w in (1, 2, 3, 4):
            if w != args.workload:
                rec = attention_record(w, dev, peaks)
                others[rec["workload"]] = rec

    # ---- attention-layer level (a "next" row): QKV and output projections (library GEMMs through
    # torch.matmul), rotary embedding on the shared layout's position ids, psa_fwd / psa_bwd, and the
    # projections' backward (paper_2410_20305_b200/layer.py); the same on the paired layout.
    layer = None
    if not args.no_layer and rank == 0:
        def layer_ms(pk_, seed):
            Tl, hid = pk_.total_tokens, Hq * d
            g = torch.Generator(device=dev); g.manual_seed(seed)
            rn = lambda *shape: (torch.randn(*shape, generator=g, device=dev) * 0.02).to(torch.bfloat16)
            x = (torch.randn(Tl, hid, generator=g, device=dev)).to(torch.bfloat16)
            dout = (torch.randn(Tl, hid, generator=g, device=dev)).to(torch.bfloat16)
            wq, wk, wv, wo = rn(hid, Hq * d), rn(hid, Hkv * d), rn(hid, Hkv * d), rn(Hq * d, hid)
            lay = AttentionLayer((pk_.cu_seqlens, pk_.prefix_len, pk_.chosen_len, pk_.rejected_len), Hq, Hkv, d, dev)

            def run():
                out, saved = lay.forward(x, wq, wk, wv, wo)
                lay.backward(x, wq, wk, wv, wo, saved, dout)
            for _ in range(3):
                run()
            torch.cuda.synchronize()
            a, b = ev(), ev()
            n_l = max(10, min(args.steps, 30))
            a.record()
            for _ in range(n_l):
                run()
            b.record()
            torch.cuda.synchronize()
            return a.elapsed_time(b) / n_l
        l_shared = layer_ms(pack, 2200 + args.workload)
        l_paired = layer_ms(pack.paired(), 2300 + args.workload)
        layer = {"hidden": Hq * d, "shared_fwd_bwd_ms": l_shared, "paired_fwd_bwd_ms": l_paired,
                 "speedup_shared_over_paired": l_paired / l_shared,
                 "projections": "torch.matmul (cuBLAS), bf16", "rope": "psa_rope on psa_position_ids"}
        torch.cuda.empty_cache()

    # ---- packing (a "next" row, host only): first-fit-decreasing over 2000 units of the workload's
    # length distribution, shared units (P + C + R) against paired units (2P + C + R), laid out for psa_plan
    packing = None
    if rank == 0:
        lens, cap = wl.sample_lengths(args.workload, 2000, 3000 + args.workload)
        lens = [(p, c, r) for p, c, r in lens if 2 * p + c + r <= cap]   # (a paired unit longer than a pack would be truncated)
        P_, C_, R_ = ([x[i] for x in lens] for i in range(3))
        t0 = time.perf_counter()
        _, packs_s = B.psa_pack_ffd_emit(P_, C_, R_, cap)
        _, packs_p = B.psa_pack_ffd_emit(P_, C_, R_, cap, paired=True)
        ms_both = (time.perf_counter() - t0) * 1e3
        tok_s = sum(int(pk["cu_seqlens"][-1]) for pk in packs_s)
        tok_p = sum(int(pk["cu_seqlens"][-1]) for pk in packs_p)
        packing = {"units": len(lens), "pack_len": cap, "packs_shared": len(packs_s), "packs_paired": len(packs_p),
                   "packs_ratio_paired_over_shared": len(packs_p) / len(packs_s), "fill_shared": tok_s / (len(packs_s) * cap),
                   "fill_paired": tok_p / (len(packs_p) * cap), "ms_both": ms_both, "call": "psa_pack_ffd_emit"}

    # ---- end to end: psa_step_host on pinned host buffers (copies in, fwd, bwd, copies out per step).
    # A few arenas, each on a stream of its own, so that one step's copies out overlap the next step's copies in
    # (the link is full duplex); a step's buffers are reused only after that step has finished.
    e2e = None
    if not args.no_e2e:
        hq, hk, hv, hdo = (t.cpu().pin_memory() for t in (q, k, v, d_o))
        h_out = [[torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in (o, lse, dq, dk, dv)] for _ in range(N_E2E)]
        h2d = sum(t.numel() * t.element_size() for t in (hq, hk, hv, hdo))
        d2h = sum(t.numel() * t.element_size() for t in h_out[0])
        arena_bytes = B.psa_step_host_arena_bytes(plan0)
        arenas = [torch.empty(arena_bytes, dtype=torch.uint8, device=dev) for _ in range(N_E2E)]
        streams = [torch.cuda.Stream(device=dev) for _ in range(N_E2E)]
        plans = []   # kept alive: freeing a plan's device blob would synchronise the device mid-pipeline

        def e2e_run(n):
            for i in range(n):
                s = i % N_E2E
                streams[s].synchronize()
                p = B.psa_plan(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len, Hq, Hkv, d,
                               stream=streams[s].cuda_stream)
                plans.append(p)
                ho = h_out[s]
                B.psa_step_host(p, hq, hk, hv, hdo, ho[0], ho[1], ho[2], ho[3], ho[4], arenas[s],
                                stream=streams[s].cuda_stream)
            for st in streams:
                st.synchronize()
        e2e_run(4)
        plans.clear()
        sync_all()
        n_e2e = max(4, min(2 * args.steps, 20))
        t0 = time.perf_counter()
        e2e_run(n_e2e)
        e2e_ms = (time.perf_counter() - t0) * 1e3 / n_e2e
        sync_all()
        plans.clear()
        # the last step's gradients, as read back on the host, must be the device path's
        # (dk is accumulated in a fixed order, hence bit-identical; dq's fp32 adds are not ordered)
        last = h_out[(n_e2e - 1) % N_E2E]
        assert torch.equal(last[3], dk.cpu()), "psa_step_host: dk differs from psa_bwd"
        assert (last[2].float() - dq.cpu().float()).abs().max().item() <= 0.0625, "psa_step_host: dq differs"
        e2e = {"value": (flops_fwd + flops_bwd) / e2e_ms / 1e9, "unit": UNIT, "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "call": "psa_step_host, %d arenas on %d streams" % (N_E2E, N_E2E), "steps": n_e2e,
               "note": "attention forward + backward through host buffers; the gather is not part of this call"}
        del arenas

    # ---- max over ranks (replicas): whole-job value = sum of the replicas' useful flops / slowest time
    step_ms, att_ms, lp_ms, e2e_ms_max = max_over_ranks(
        [step_ms, att_ms, lp_ms, e2e["ms_per_step"] if e2e else 0.0], dev)
    flops_all, tokens_all = sum_over_ranks([flops_fwd + flops_bwd, float(T)], dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    if all_rows:
        all_rows["frac_of_hbm"] = {"measured": all_rows["gbs"] / peaks["hbm_gbs"], "nominal": all_rows["gbs"] / NOMINAL_HBM_GBS}
    value = whole_job_tflops(flops_all, att_ms)
    att_min_bytes = T * (6 * Hq + 6 * Hkv) * d * 2
    bwd_ms, fwd_ms, klp_ms = kernel_ms["bwd"], kernel_ms["fwd"], kernel_ms["logp"]
    # A region of half a second or more runs under the power cap at a reduced SM clock: the peak to
    # read it against is the sustained one (a cuBLAS loop of seconds); a short region against the burst.
    sustained = timed_ms >= 400.0 and peaks.get("bf16_tflops_sustained")
    peak_tc = peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"]
    peak_kind = ("sustained" if sustained else "burst") + " bf16 cuBLAS, of " + peaks["source"]
    bwd_tflops = flops_bwd / bwd_ms / 1e9
    logp_bytes = live_rows * VOCAB * 2 + 8 * live_rows + 4 * n_seg
    clk = clocks.summary()
    sm_mhz = clk.get("sm_mhz")
    traffic, traffic_note = ncu_traffic("psa_bwd_kernel", pack.name)
    frac_meas, frac_nom = value / world / peaks["bf16_tflops"], value / world / NOMINAL_BF16_TFLOPS
    frac_sus = value / world / peaks["bf16_tflops_sustained"] if peaks.get("bf16_tflops_sustained") else None
    logp_frac_meas = logp_bytes / klp_ms / 1e6 / peaks["hbm_gbs"] if not args.no_logp else None
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": pack.name, "pack_len": pack.pack_len, "total_tokens": T, "n_samples": pack.n_samples,
                   "n_q_heads": Hq, "n_kv_heads": Hkv, "head_dim": d, "useful_pairs_per_head": U,
                   "live_tiles": plan0.live_tiles, "partial_tiles": plan0.partial_tiles, "logits": [T, VOCAB],
                   "l2": "inputs larger than L2 (q, o, dO, dq are %.0f MB each; logits %.1f GB)" % (T * Hq * d * 2 / 1e6, T * VOCAB * 2 / 1e9),
                   "parallelism": ("one pack per GPU (%d packs, %d tokens in all; rank 0's pack is described here), "
                                   "no collective on the data path" % (world, int(tokens_all))) if world > 1 else "single GPU"},
        "inner_repeats": inner,
        "timed_region": {"passes": n_pass, "ms": timed_ms,
                         "note": "each of the --steps steps is run inner_repeats times so that the region lasts at least "
                                 "%.1f s; every figure is per pass" % MIN_TIMED_SECONDS},
        "attention_fwd_bwd_ms": att_ms,
        "attention_fwd_bwd_ms_median_min": [float(np.median(att_all)), float(np.min(att_all))],
        # duration x clock: what the same work would cost at another SM clock (the part is power-limited under
        # tensor load; NVML's samples are the only clock reading a program can take without touching any setting)
        "attention_fwd_bwd_ms_x_sm_mhz": att_ms * sm_mhz if sm_mhz else None,
        "plan_ms_host": plan_host_ms,
        "plan_ms_host_per_layer_of_32": plan_host_ms / 32,   # one plan serves every layer of a step
        "pct_of_bf16_peak": {"measured": frac_meas, "measured_sustained": frac_sus, "nominal": frac_nom,
                             "peak_source": peaks["source"],
                             "note": "measured = burst cuBLAS rate (%.1f), measured_sustained = the same GEMM looped for "
                                     "seconds under the power cap (%s); the timed region here lasts %.2f s"
                                     % (peaks["bf16_tflops"], peaks.get("bf16_tflops_sustained"), timed_ms * 1e-3)},
        "target": {"attention_fwd_bwd_frac_of_bf16_peak": TARGET_FRAC_OF_BF16_PEAK,
                   "met_against_measured_peak": bool(frac_meas >= TARGET_FRAC_OF_BF16_PEAK),
                   "met_against_measured_sustained_peak": None if frac_sus is None else bool(frac_sus >= TARGET_FRAC_OF_BF16_PEAK),
                   "met_against_nominal_peak": bool(frac_nom >= TARGET_FRAC_OF_BF16_PEAK),
                   "gather_frac_of_hbm": TARGET_FRAC_OF_HBM,
                   "gather_met_against_measured": None if logp_frac_meas is None else bool(logp_frac_meas >= TARGET_FRAC_OF_HBM),
                   "gather_met_against_nominal": None if logp_frac_meas is None else
                   bool(logp_bytes / klp_ms / 1e6 / NOMINAL_HBM_GBS >= TARGET_FRAC_OF_HBM)},
        # the other bound of attention fwd+bwd: six passes over Hq-sized and six over Hkv-sized tensors
        # (the short-many workload sits below the ridge point and is bounded by this one)
        "attention_min_hbm": {"bytes": att_min_bytes, "gbs": att_min_bytes / att_ms / 1e6,
                              "frac_of_hbm": {"measured": att_min_bytes / att_ms / 1e6 / peaks["hbm_gbs"],
                                              "nominal": att_min_bytes / att_ms / 1e6 / NOMINAL_HBM_GBS}},
        "tokens_per_s": tokens_all / (step_ms * 1e-3),
        "attention_tokens_per_s": tokens_all / (att_ms * 1e-3),
        "kernels": {"psa_fwd_ms": fwd_ms, "psa_fwd_tflops": flops_fwd / fwd_ms / 1e9,
                    "psa_fwd_frac_of_measured_peak": flops_fwd / fwd_ms / 1e9 / peaks["bf16_tflops"],
                    "psa_bwd_main_ms": bwd_ms, "psa_bwd_main_tflops": bwd_tflops,
                    "psa_bwd_delta_clear_ms": kernel_ms["bwd_delta_clear"], "psa_bwd_convert_ms": kernel_ms["bwd_convert"],
                    "timing": "CUDA events recorded by the library around each kernel, every pass of the timed region",
                    "dpo_logp_ms": klp_ms, "dpo_logp_gbs": logp_bytes / klp_ms / 1e6,
                    "dpo_logp_frac_of_hbm": {"measured": logp_bytes / klp_ms / 1e6 / peaks["hbm_gbs"],
                                             "nominal": logp_bytes / klp_ms / 1e6 / NOMINAL_HBM_GBS},
                    "dpo_logp_live_rows": live_rows, "dpo_logp_step_ms": lp_ms},
        "roofline": {"kernel": "psa_bwd_kernel<%d>" % d, "bound": "tensor", "achieved": bwd_tflops,
                     "peak": peak_tc, "unit": "TFLOP/s", "frac": bwd_tflops / peak_tc,
                     "frac_of_burst_peak": bwd_tflops / peaks["bf16_tflops"],
                     "scope": "this one kernel (the dominant one), not the attention forward + backward as a whole: "
                              "that is pct_of_bf16_peak",
                     "peak_kind": peak_kind,
                     "algorithmic_flops": flops_bwd, "algorithmic_bytes": T * (4 * Hq + 4 * Hkv) * d * 2,
                     "traffic": traffic, "traffic_source": traffic_note},
        "clocks": clk,
        "gpu_launches": n_pass * (4 if args.no_logp else 5),
        "paired_layout": paired,
        "workloads": others,
        "dpo_logp_all_rows": all_rows,
        "next_rows": loss_bwd,
        "attention_layer": layer,
        "packing": packing,
        "paper_context": "paper reports 1.1-1.5x (1.3-1.6x with packing) end-to-end training speedups on 8xH100; context, not the target",
    }
    if e2e:
        e2e["value"] = whole_job_tflops(flops_all, e2e_ms_max)
        e2e["ms_per_step"] = e2e_ms_max
        line["e2e"] = e2e
    if not args.no_cpu_baseline and world == 1:
        # two untimed and eight timed passes over the sample: about 15 s of host work
        val, desc, cores, sec = oracle_sample(pack, 8, 2)
        line["cpu_baseline"] = {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc,
                                "seconds_per_pass": sec, "timed_passes": 8}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
