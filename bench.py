#!/usr/bin/env python
"""Benchmark of the prefix-shared DPO hot path on B200.

One "step" is one pass of the whole path over one synthetic pack: psa_plan on the
host, psa_fwd, psa_bwd, and dpo_logp over the pack's logits.  The headline metric
is the useful TFLOP/s of attention forward + backward (14*d*Hq*U flops, U = the
unmasked (q, kv) pairs per head) over the time of those two calls, measured with
CUDA events inside the timed steps; packed tokens/s over the whole step and the
gather's GB/s are reported beside it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 1..4] [--impl reference]

N > 1 (launched through torch.distributed.run) runs N independent replicas: the
path has no exchange step, so there is no collective on the data path.
"""
from __future__ import annotations

import argparse
import json
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
# DRAM bytes (read + write) of one psa_bwd_kernel launch, from the ncu capture summarised in
# profiles/psa_bwd_kernel_llama3-8b.md (workload 1); other workloads have no capture.
N_E2E = int(os.environ.get("PSA_BENCH_E2E_STREAMS", "3"))   # arenas / streams of the end-to-end leg
NCU_BWD_TRAFFIC_BYTES = {1: 1454.7e6}


def measured_peaks():
    """Roofline denominators: the measured copy bandwidth and cuBLAS bf16 rate of
    this machine's B200s if the driver left them, else an earlier measurement."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


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
                    "sm_max_mhz": self.max_sm, "reasons": reasons, "samples": len(self.sm), "source": "nvml, every 2 ms",
                    "note": "NVML's reading; inside the attention kernels ncu's sm__cycles_elapsed.avg.per_second is "
                            "1.59-1.68 GHz (see profiles/), with no clock-event reason raised"}
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


def whole_job_tflops(flops_per_replica, world, ms):
    """N independent replicas: the job's work is the sum, its time the slowest rank's."""
    return world * flops_per_replica / ms / 1e9


def oracle_sample(pack, steps, warmup, target="bench"):
    """Times the fp64 oracle, as it stands, on a bounded sample of the workload: whole
    samples of the pack (attention is independent per sample, which the oracle's own tests
    pin) for one kv group of 4 query heads.  The baseline leg takes every sample of the
    pack (1/8 of the workload's heads), the reference arm only the shortest sample because
    it runs many steps.  Returns (useful TFLOP/s, description, cores, seconds per step)."""
    import torch
    from oracle import psa_oracle as orc
    from paper_2410_20305_b200 import workloads as wl
    order = np.argsort(pack.cu_seqlens[1:] - pack.cu_seqlens[:-1])
    chosen = [int(x) for x in (order if target == "bench" else order[:1])]
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
    desc = "%d sample(s) of the pack (%d tokens), 4 query heads / 1 kv head, fwd+bwd, dense fp64 numpy" % (
        len(chosen), int(sum(pack.cu_seqlens[s + 1] - pack.cu_seqlens[s] for s in chosen)))
    return flops / sec / 1e12, desc, torch.get_num_threads(), sec


def run_reference(args, pack, rank):
    """The reference arm: the CPU oracle on the machine's host cores, rank 0 only."""
    if rank != 0:
        return
    val, desc, cores, sec = oracle_sample(pack, args.steps, args.warmup, target="reference")
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": pack.name, "sample": desc},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="psa", choices=["psa", "reference"])
    ap.add_argument("--workload", type=int, default=1, help="1 llama3-8b, 2 long-prompt, 3 multi-turn, 4 short-many")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-layer", action="store_true")
    ap.add_argument("--no-paired", action="store_true")
    ap.add_argument("--no-logp", action="store_true", help="attention only (small footprint, for ncu captures)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    from paper_2410_20305_b200 import workloads as wl
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    pack = wl.config_pack(args.workload)
    if args.impl == "reference":
        return run_reference(args, pack, rank)

    import torch
    import torch.distributed as dist
    import paper_2410_20305_b200 as psa
    from paper_2410_20305_b200 import binding as B

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

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
    n_total = args.warmup + args.steps
    e_att0, e_att1, e_lp1 = [ev() for _ in range(n_total)], [ev() for _ in range(n_total)], [ev() for _ in range(n_total)]
    k_fwd, k_bwd, k_lp = (ev(), ev()), (ev(), ev()), (ev(), ev())
    kernel_ms = {"fwd": [], "bwd": [], "logp": []}

    def step(i, timed):
        plan = B.psa_plan(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len, Hq, Hkv, d)
        e_att0[i].record()
        B.psa_fwd(plan, q, k, v, o=o, lse=lse, status=status)
        B.psa_bwd(plan, d_o, q, k, v, o, lse, dq=dq, dk=dk, dv=dv, workspace=ws, status=status)
        e_att1[i].record()
        if not args.no_logp:
            B.dpo_logp(logits, targets, seg_d, n_seg, fr, ft, fs, out=logp, status=status)
        e_lp1[i].record()
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

    # Per-kernel events (the library records them right around each main kernel) are read one
    # step at a time in a separate short pass so that the timed region below stays free of syncs.
    for i in range(args.warmup):
        step(i, False)
    sync_all()
    for name, which, pair in (("fwd", 0, k_fwd), ("bwd", 1, k_bwd), ("logp", 2, k_lp)):
        B.psa_profile_events(which, *pair)
    for i in range(min(args.steps, 10)):
        step(0, False)
        torch.cuda.synchronize()
        for name, pair in (("fwd", k_fwd), ("bwd", k_bwd), ("logp", k_lp)):
            if name == "logp" and args.no_logp:
                kernel_ms[name].append(float("nan"))
            else:
                kernel_ms[name].append(pair[0].elapsed_time(pair[1]))
    for which in range(3):
        B.psa_profile_events(which)

    sync_all()
    t_start, t_stop = ev(), ev()
    with ClockSampler(local_rank) as clocks:
        t_start.record()
        for i in range(args.warmup, n_total):
            step(i, True)
        t_stop.record()
        sync_all()
    step_ms = t_start.elapsed_time(t_stop) / args.steps
    att_all = [e_att0[i].elapsed_time(e_att1[i]) for i in range(args.warmup, n_total)]
    att_ms = float(np.mean(att_all))
    lp_ms = float(np.mean([e_att1[i].elapsed_time(e_lp1[i]) for i in range(args.warmup, n_total)]))
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
        a.record()
        for _ in range(args.steps):
            B.psa_fwd(pplan, pq, pk, pv, o=po, lse=plse)
            B.psa_bwd(pplan, pdo, pq, pk, pv, po, plse, dq=pdq, dk=pdk, dv=pdv, workspace=pws)
        b.record()
        torch.cuda.synchronize()
        p_ms = a.elapsed_time(b) / args.steps
        paired = {"tokens": pp.total_tokens, "fwd_bwd_ms": p_ms, "speedup_shared_over_paired": p_ms / att_ms,
                  "ideal_pair_ratio": pplan.useful_pairs / U, "token_ratio": pp.total_tokens / T}
        del pq, pk, pv, pdo, po, plse, pws, pdq, pdk, pdv

    # ---- attention-layer level (a "next" row): QKV and output projections (library GEMMs through
    # torch.matmul), rotary embedding on the shared layout's position ids, psa_fwd / psa_bwd, and the
    # projections' backward; the same on the paired layout.
    layer = None
    if not args.no_layer and rank == 0:
        def layer_ms(pk_, seed):
            Tl = pk_.total_tokens
            hid = Hq * d
            g = torch.Generator(device=dev); g.manual_seed(seed)
            rn = lambda *shape: (torch.randn(*shape, generator=g, device=dev) * 0.02).to(torch.bfloat16)
            x = (torch.randn(Tl, hid, generator=g, device=dev)).to(torch.bfloat16)
            dout = (torch.randn(Tl, hid, generator=g, device=dev)).to(torch.bfloat16)
            wq, wk, wv, wo = rn(hid, Hq * d), rn(hid, Hkv * d), rn(hid, Hkv * d), rn(Hq * d, hid)
            pos = torch.as_tensor(B.psa_position_ids(pk_.cu_seqlens, pk_.prefix_len, pk_.chosen_len, pk_.rejected_len)).to(dev)
            neg = -pos
            lplan = B.psa_plan(pk_.cu_seqlens, pk_.prefix_len, pk_.chosen_len, pk_.rejected_len, Hq, Hkv, d)
            lws = torch.empty(lplan.bwd_workspace_bytes, dtype=torch.uint8, device=dev)

            def run():
                q_ = (x @ wq).view(Tl, Hq, d); k_ = (x @ wk).view(Tl, Hkv, d); v_ = (x @ wv).view(Tl, Hkv, d)
                B.psa_rope(q_, pos, out=q_); B.psa_rope(k_, pos, out=k_)
                o_, lse_ = B.psa_fwd(lplan, q_, k_, v_)
                out = o_.view(Tl, hid) @ wo                                   # noqa: F841  (the layer's output)
                do_ = (dout @ wo.t()).view(Tl, Hq, d)
                dwo = o_.view(Tl, hid).t() @ dout                             # noqa: F841
                dq_, dk_, dv_ = B.psa_bwd(lplan, do_, q_, k_, v_, o_, lse_, workspace=lws)
                B.psa_rope(dq_, neg, out=dq_); B.psa_rope(dk_, neg, out=dk_)   # gradient of a rotation: the inverse rotation
                dq2, dk2, dv2 = dq_.view(Tl, -1), dk_.view(Tl, -1), dv_.view(Tl, -1)
                dx = dq2 @ wq.t() + dk2 @ wk.t() + dv2 @ wv.t()               # noqa: F841
                dwq, dwk, dwv = x.t() @ dq2, x.t() @ dk2, x.t() @ dv2         # noqa: F841
            for _ in range(3):
                run()
            torch.cuda.synchronize()
            a, b = ev(), ev()
            a.record()
            for _ in range(args.steps):
                run()
            b.record()
            torch.cuda.synchronize()
            return a.elapsed_time(b) / args.steps
        l_shared = layer_ms(pack, 2200 + args.workload)
        l_paired = layer_ms(pack.paired(), 2300 + args.workload)
        layer = {"hidden": Hq * d, "shared_fwd_bwd_ms": l_shared, "paired_fwd_bwd_ms": l_paired,
                 "speedup_shared_over_paired": l_paired / l_shared,
                 "projections": "torch.matmul (cuBLAS), bf16", "rope": "psa_rope on psa_position_ids"}
        torch.cuda.empty_cache()

    # ---- packing (a "next" row, host only): first-fit-decreasing over 2000 units of the workload's
    # length distribution, shared units (P + C + R) against paired units (2P + C + R)
    packing = None
    if rank == 0:
        lens, cap = wl.sample_lengths(args.workload, 2000, 3000 + args.workload)
        shared = [p + c + r for p, c, r in lens]
        paired_u = [min(2 * p + c + r, cap) for p, c, r in lens]   # (a unit longer than a pack would be truncated)
        t0 = time.perf_counter()
        _, nb_s = B.psa_pack_ffd(shared, cap)
        _, nb_p = B.psa_pack_ffd(paired_u, cap)
        packing = {"units": len(lens), "pack_len": cap, "packs_shared": nb_s, "packs_paired": nb_p,
                   "packs_ratio_paired_over_shared": nb_p / nb_s, "fill_shared": sum(shared) / (nb_s * cap),
                   "fill_paired": sum(paired_u) / (nb_p * cap), "ms_both": (time.perf_counter() - t0) * 1e3}

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
               "call": "psa_step_host, %d arenas on %d streams" % (N_E2E, N_E2E), "steps": n_e2e}
        del arenas

    # ---- max over ranks (replicas): whole-job value = sum of the replicas' useful flops / slowest time
    step_ms, att_ms, lp_ms, e2e_ms_max = max_over_ranks(
        [step_ms, att_ms, lp_ms, e2e["ms_per_step"] if e2e else 0.0], dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    if all_rows:
        all_rows["frac_of_hbm"] = {"measured": all_rows["gbs"] / peaks["hbm_gbs"], "nominal": all_rows["gbs"] / NOMINAL_HBM_GBS}
    value = whole_job_tflops(flops_fwd + flops_bwd, world, att_ms)
    att_min_bytes = T * (6 * Hq + 6 * Hkv) * d * 2
    bwd_ms, fwd_ms, klp_ms = (float(np.mean(kernel_ms[n])) for n in ("bwd", "fwd", "logp"))
    bwd_tflops = flops_bwd / bwd_ms / 1e9
    logp_bytes = live_rows * VOCAB * 2 + 8 * live_rows + 4 * n_seg
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": pack.name, "pack_len": pack.pack_len, "total_tokens": T, "n_samples": pack.n_samples,
                   "n_q_heads": Hq, "n_kv_heads": Hkv, "head_dim": d, "useful_pairs_per_head": U,
                   "live_tiles": plan0.live_tiles, "partial_tiles": plan0.partial_tiles, "logits": [T, VOCAB],
                   "l2": "inputs larger than L2 (q, o, dO, dq are 133 MB each; logits %.1f GB)" % (T * VOCAB * 2 / 1e9),
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "attention_fwd_bwd_ms": att_ms,
        "attention_fwd_bwd_ms_median_min": [float(np.median(att_all)), float(np.min(att_all))],
        "plan_ms_host": plan_host_ms,
        "plan_ms_host_per_layer_of_32": plan_host_ms / 32,   # one plan serves every layer of a step
        "pct_of_bf16_peak": {"measured": value / world / peaks["bf16_tflops"], "nominal": value / world / NOMINAL_BF16_TFLOPS,
                             "peak_source": peaks["source"]},
        # the other bound of attention fwd+bwd: six passes over Hq-sized and six over Hkv-sized tensors
        # (the short-many workload sits below the ridge point and is bounded by this one)
        "attention_min_hbm": {"bytes": att_min_bytes, "gbs": att_min_bytes / att_ms / 1e6,
                              "frac_of_hbm": {"measured": att_min_bytes / att_ms / 1e6 / peaks["hbm_gbs"],
                                              "nominal": att_min_bytes / att_ms / 1e6 / NOMINAL_HBM_GBS}},
        "tokens_per_s": world * T / (step_ms * 1e-3),
        "attention_tokens_per_s": world * T / (att_ms * 1e-3),
        "kernels": {"psa_fwd_ms": fwd_ms, "psa_fwd_tflops": flops_fwd / fwd_ms / 1e9,
                    "psa_bwd_main_ms": bwd_ms, "psa_bwd_main_tflops": bwd_tflops,
                    "dpo_logp_ms": klp_ms, "dpo_logp_gbs": logp_bytes / klp_ms / 1e6,
                    "dpo_logp_frac_of_hbm": {"measured": logp_bytes / klp_ms / 1e6 / peaks["hbm_gbs"],
                                             "nominal": logp_bytes / klp_ms / 1e6 / NOMINAL_HBM_GBS},
                    "dpo_logp_live_rows": live_rows, "dpo_logp_step_ms": lp_ms},
        "roofline": {"kernel": "psa_bwd_kernel<128>", "bound": "tensor", "achieved": bwd_tflops,
                     "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": bwd_tflops / peaks["bf16_tflops"],
                     "peak_kind": "burst bf16 cuBLAS, of " + peaks["source"],
                     "algorithmic_flops": flops_bwd, "algorithmic_bytes": 40960.0 * T if (Hq, Hkv, d) == (32, 8, 128) else None,
                     "traffic": NCU_BWD_TRAFFIC_BYTES.get(args.workload)},
        "clocks": clocks.summary(),
        "gpu_launches": args.steps * (4 if args.no_logp else 5),
        "paired_layout": paired,
        "dpo_logp_all_rows": all_rows,
        "next_rows": loss_bwd,
        "attention_layer": layer,
        "packing": packing,
        "paper_context": "paper reports 1.1-1.5x (1.3-1.6x with packing) end-to-end training speedups on 8xH100; context, not the target",
    }
    if e2e:
        e2e["value"] = whole_job_tflops(flops_fwd + flops_bwd, world, e2e_ms_max)
        e2e["ms_per_step"] = e2e_ms_max
        line["e2e"] = e2e
    if not args.no_cpu_baseline and world == 1:
        # one untimed and three timed passes over the sample: about 13 s of host work on workload 1
        val, desc, cores, sec = oracle_sample(pack, 3, 1)
        line["cpu_baseline"] = {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc,
                                "seconds_per_pass": sec, "timed_passes": 3}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
