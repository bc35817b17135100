#!/usr/bin/env python
"""Benchmark of the CAT loss hot path (fused LM head + CAT-weighted cross-entropy, fwd + bwd).

One step = the whole hot path, forward and backward (one cat_loss_fwd_bwd call), over one synthetic
draft-training batch of the Llama-3.2-1B-shaped head config (T=16384 rows in blocks of K=8, d=2048,
V=128256, bf16); the two-call form (cat_loss_fwd + cat_loss_bwd, logits recomputed) is timed beside it.
Prints ONE JSON line.  `value` is tokens/s with inputs resident in HBM; `e2e` is the same
metric with host (pinned) buffers, host<->device copies inside the timed region; `roofline`
is the GEMM with the largest share of the step, timed by events inside the timed steps, against
the measured dense bf16 peak (`stages` has every stage; `roofline_fwd_two_call` the forward GEMM
of the two-call path);
`cpu_baseline` is the fp64 oracle timed on this machine's host cores on a bounded sample.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 2]
For N > 1 launch with torch.distributed.run; ranks run independent batches (draft blocks are
independent, so the path shards by rows with no data-path collective: weak scaling).
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch

# dram__bytes_read.sum + dram__bytes_write.sum of ONE launch of a kernel (CTA-pair build) on the bench
# workload, from the ncu captures summarised in profiles/ (ncu_full_fused_gemms_config2.md for the
# first row slab of the one-call path, ncu_two_call_gemms_config2.md for the two-call forward).
# Valid for that kernel, workload and T only; None for anything else.
TRAFFIC_BYTES = {
    ("config2", 16384, "logits"): 972038000 + 2392758000,
    ("config2", 16384, "dH"): 8332829000 + 36699000,
    ("config2", 16384, "dW"): 4663208000 + 1036382000,
    ("config2", 16384, "fwd_two_call"): 3061464832 + 21341440,
}
STAGES = ("label_ref", "logits", "rows", "slab_prep", "dH", "dW")
STAGE_KERNEL = {
    "logits": "tc::gemm_kernel<K-major,K-major,EpiFwdExp,pair> logits + softmax partials + bf16 exp(z - ref) store",
    "dH": "tc::gemm_kernel<K-major,MN-major,EpiOut,pair> dH slab = dz W",
    "dW": "tc::gemm_kernel<MN-major,MN-major,EpiOut,pair> dW += dz^T H",
}

METRIC = "cat_loss_fwd_bwd_tokens_per_s"
UNIT = "tokens/s"


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return dict(burst=float(j["bf16_tflops"]), sustained=float(j["bf16_tflops_sustained"]), hbm=float(j["hbm_gbs"]),
                    source="measured")
    return dict(burst=1590.0, sustained=1400.0, hbm=6650.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index):
        self.idx, self.rows, self.proc = device_index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.idx)], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.25)
        self.proc.terminate()
        sm = [float(r[1]) for r in self.rows if len(r) >= 9 and r[1].replace(".", "").isdigit()]
        mx = [float(r[2]) for r in self.rows if len(r) >= 9 and r[2].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = set()
        for r in self.rows:
            if len(r) >= 9:
                for n, v in zip(names, r[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


def oracle_sample_rate(batch, rows, steps=1):
    """tokens/s of the fp64 oracle (fwd + bwd, incl. those rows' dW contribution) on the first `rows` rows."""
    from oracle import cat_oracle as O
    H, y, v = batch.H[:rows], batch.labels[:rows], batch.valid[:rows]
    Hd, Wd = H.double().numpy(), batch.W.double().numpy()
    times = []
    for _ in range(steps):
        t0 = time.perf_counter()
        O.cat_forward_backward(Hd, Wd, y, v, batch.K, row_chunk=256)
        times.append(time.perf_counter() - t0)
    return rows / (sum(times) / len(times)), sum(times) / len(times) * 1e3


def host_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p["num_threads"] for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2)
    ap.add_argument("--rows", type=int, default=0, help="override T (debug / profiling of a small case)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the Eq. 12 (cross-entropy + distillation) timing")
    ap.add_argument("--profile", choices=["fused", "two-call", "kd"], default=None,
                    help="run only that path for --warmup + --steps steps and exit (for ncu captures of a small case; prints no bench line)")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    from paper_2605_08632_b200 import synth
    spec = synth.CONFIGS[args.config]
    T = args.rows if args.rows else spec.T
    cfg = dict(workload=f"config{args.config}:{spec.name}", T=T, K=spec.K, d=spec.d, V=spec.V, rows_per_gpu=T,
               labels=spec.labels, l2="inputs larger than L2 (W alone is %.0f MB)" % (spec.V * spec.d * 2 / 1e6),
               parallelism=f"rows sharded by whole draft blocks x{args.gpus}, no collective")
    flops_per_token = 6.0 * spec.d * spec.V

    # ------------------------------------------------------------------ reference arm: the oracle on host cores
    if args.impl == "reference":
        if rank != 0:
            return
        batch = synth.make_batch(args.config, T=min(T, 2048))
        rows = 256
        for _ in range(max(0, min(args.warmup, 1))):
            oracle_sample_rate(batch, rows)
        rate, ms = oracle_sample_rate(batch, rows, steps=max(1, args.steps))
        cores = host_threads()
        print(json.dumps({
            "impl": "reference", "metric": METRIC, "value": rate, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "config": cfg,
            "cpu_baseline": {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"{rows} rows (whole K-blocks) of the workload per step, fwd+bwd incl. their dW contribution"},
            "e2e": {"value": rate, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}))
        return

    # ------------------------------------------------------------------ our arm
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path for the product")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    from paper_2605_08632_b200.api import CatLoss
    from paper_2605_08632_b200 import binding as B

    batch = synth.make_batch(args.config, T=T)
    if world > 1:   # every rank its own rows: re-draw H and labels with a rank-dependent seed
        g = torch.Generator().manual_seed(1000 + rank)
        batch.H = torch.randn(T, spec.d, generator=g).to(batch.torch_dtype)
        batch.labels = torch.randint(0, spec.V, (T,), generator=g)
    H, W = batch.H.to(dev), batch.W.to(dev)
    labels, valid = batch.labels.to(dev), batch.valid.to(dev)
    cl = CatLoss(T, spec.d, spec.V, spec.K, dtype=batch.torch_dtype)

    def step():
        cl.forward_backward(H, W, labels, valid)

    def step_split():
        cl.forward(H, W, labels, valid)
        cl.backward(H, W, labels, valid)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def reduce_max(ms):
        if world > 1:
            t = torch.tensor([ms], device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            return float(t.item())
        return ms

    def kd_setup():
        # Eq. 12 on the same batch: a Llama-3.1-8B-shaped target head (d_t = 4096) over the
        # T/K + K - 1 sequence positions the batch's blocks refer to, beta = 0.1
        ts = synth.make_target_side(batch, d_t=4096)
        Ht, Wt = ts.Ht.to(dev), ts.Wt.to(dev)
        return ts, (lambda: cl.kd_forward_backward(H, W, labels, valid, Ht, Wt, ts.block_start, 0.1))

    if args.profile:
        fn = {"fused": step, "two-call": step_split}.get(args.profile) or kd_setup()[1]
        for _ in range(args.warmup + args.steps):
            fn()
        torch.cuda.synchronize()
        print(json.dumps({"profile_run": args.profile, "T": T, "note": "not a benchmark value"}))
        return

    stream = torch.cuda.current_stream()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    # ---- headline: the fused call (cat_loss_fwd_bwd: logits kept per row slab, 6*T*d*V executed)
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    barrier()
    # the timed steps go through cat_loss_fwd_bwd_events: the same kernels, plus an event recorded between
    # stages, so that every kernel of the step is timed inside the timed region itself
    stage_events = []
    ev0.record(stream)
    for i in range(args.steps):
        stage_events.append(cl.forward_backward_timed(H, W, labels, valid) if spec.dtype == "bf16" else step())
    ev1.record(stream)
    barrier()
    clocks = sampler.stop()
    total_ms = reduce_max(ev0.elapsed_time(ev1))
    ms_per_step = total_ms / args.steps
    value = world * T / (ms_per_step * 1e-3)
    assert cl.fwd_stats().device_status == 0 and cl.fused_status() == 0, "device reported a timed-out wait"

    # ---- the two-call path (cat_loss_fwd + cat_loss_bwd, logits recomputed: 8*T*d*V executed); the forward
    #      GEMM launch is bracketed by events on the launching stream for the roofline entry
    for _ in range(3):
        step_split()
    fwd_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    barrier()
    ev0.record(stream)
    for i in range(args.steps):
        fwd_ev[i][0].record(stream)
        cl.forward(H, W, labels, valid)
        fwd_ev[i][1].record(stream)
        cl.backward(H, W, labels, valid)
    ev1.record(stream)
    barrier()
    split_ms = reduce_max(ev0.elapsed_time(ev1)) / args.steps
    fwd_ms = statistics.mean(a.elapsed_time(b) for a, b in fwd_ev)
    assert cl.fwd_stats().device_status == 0 and cl.bwd_status() == 0, "device reported a timed-out wait"

    # ---- Eq. 12 (CAT-weighted cross-entropy + distillation): four contractions, one of them on the target side
    kd_info = None
    if not args.no_extras and world == 1:
        ts, kd_step = kd_setup()
        for _ in range(3):
            kd_step()
        kd_steps = max(2, min(args.steps, 5))
        barrier()
        ev0.record(stream)
        for _ in range(kd_steps):
            kd_step()
        ev1.record(stream)
        barrier()
        kd_ms = ev0.elapsed_time(ev1) / kd_steps
        assert cl.kd_status() == 0, "device reported a timed-out wait"
        kd_flops = 6.0 * T * spec.d * spec.V + 2.0 * ts.L * ts.d_t * spec.V
        kd_info = {"what": "cat_kd_loss_fwd_bwd (Eq. 12): draft head as the workload, target head d_t=4096 over L=%d positions, beta=0.1" % ts.L,
                   "ms_per_step": kd_ms, "value": T / (kd_ms * 1e-3), "unit": UNIT, "tflops_executed": kd_flops / (kd_ms * 1e-3) / 1e12,
                   "steps": kd_steps}
        del ts, kd_step
        cl._ws_kd = None
        torch.cuda.empty_cache()

    # ------------------------------------------------------------------ end to end with host buffers
    e2e = None
    if not args.no_e2e:
        Hh, Wh = batch.H.pin_memory(), batch.W.pin_memory()
        yh, vh = batch.labels.pin_memory(), batch.valid.pin_memory()
        loss_h = torch.empty(1, dtype=torch.float32).pin_memory()
        dH_h = torch.empty(T, spec.d, dtype=batch.torch_dtype).pin_memory()
        dW_h = torch.empty(spec.V, spec.d, dtype=torch.float32).pin_memory()

        # Two slots of device inputs and outputs, three streams: while step i computes, the inputs of step
        # i+1 arrive and the results of step i-1 leave.  Every step still copies its own inputs from pinned
        # host memory and its own results (loss, dH, dW) back; the copies overlap other steps' compute.
        cls = [cl, CatLoss(T, spec.d, spec.V, spec.K, dtype=batch.torch_dtype)]
        ins = [(H, W, labels, valid), tuple(torch.empty_like(x) for x in (H, W, labels, valid))]
        s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
        in_ready = [torch.cuda.Event() for _ in range(2)]
        comp_done = [torch.cuda.Event() for _ in range(2)]
        out_done = [torch.cuda.Event() for _ in range(2)]
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

        def e2e_step(i):
            k = i & 1
            c, (Hd, Wd, yd, vd) = cls[k], ins[k]
            with torch.cuda.stream(s_in):
                s_in.wait_event(comp_done[k])            # the slot's previous step has read its inputs
                Hd.copy_(Hh, non_blocking=True); Wd.copy_(Wh, non_blocking=True)
                yd.copy_(yh, non_blocking=True); vd.copy_(vh, non_blocking=True)
                in_ready[k].record(s_in)
            stream.wait_event(in_ready[k])
            stream.wait_event(out_done[k])               # the slot's previous results have left
            c.forward_backward(Hd, Wd, yd, vd)
            comp_done[k].record(stream)
            with torch.cuda.stream(s_out):
                s_out.wait_event(comp_done[k])
                loss_h.copy_(c.loss, non_blocking=True); dH_h.copy_(c.dH, non_blocking=True); dW_h.copy_(c.dW, non_blocking=True)
                out_done[k].record(s_out)

        e2e_steps = max(4, min(args.steps, 10))
        for k in range(2):
            comp_done[k].record(stream); out_done[k].record(stream)
        e2e_step(0); e2e_step(1)
        barrier()
        t0.record(s_in)
        for i in range(e2e_steps):
            e2e_step(i)
        with torch.cuda.stream(s_out):
            t1.record(s_out)
        barrier()
        e_ms = reduce_max(t0.elapsed_time(t1))
        assert all(c.fused_status() == 0 for c in cls), "device reported a timed-out wait"
        h2d = sum(x.numel() * x.element_size() for x in (Hh, Wh, yh, vh))
        d2h = sum(x.numel() * x.element_size() for x in (loss_h, dH_h, dW_h))
        e2e = {"value": world * T / (e_ms / e2e_steps * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": e_ms / e2e_steps,
               "how": "cat_loss_fwd_bwd through the binding; per step H2D of H, W, labels, valid from pinned memory and D2H of "
                      "loss, dH, dW, double-buffered so that copies overlap the neighbouring steps' compute"}
        del cls, ins
        torch.cuda.empty_cache()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    fwd_flops = 2.0 * T * spec.d * spec.V
    achieved = fwd_flops / (fwd_ms * 1e-3) / 1e12
    pair = os.environ.get("CAT_LOSS_CTA_PAIR", "1") != "0"

    # per-stage device times of the one-call path inside the timed region (averages over the timed steps)
    stage_info, roofline = None, None
    if spec.dtype == "bf16":
        slabs = B.cat_loss_fused_slabs(cl.shape)
        n_slabs = len(slabs) - 1
        per = {st: [0.0] * n_slabs for st in STAGES}
        other = 0.0
        for evs in stage_events:
            other += evs[0].elapsed_time(evs[1]) + evs[-2].elapsed_time(evs[-1])
            for sl in range(n_slabs):
                for j, st in enumerate(STAGES):
                    per[st][sl] += evs[1 + len(STAGES) * sl + j].elapsed_time(evs[2 + len(STAGES) * sl + j])
        for st in STAGES:
            per[st] = [x / args.steps for x in per[st]]
        stage_info = {"slab_rows": [slabs[i + 1] - slabs[i] for i in range(n_slabs)],
                      "ms_per_launch": per, "ms_per_step": {st: sum(per[st]) for st in STAGES},
                      "other_ms_per_step": other / args.steps}
        # the roofline entry is the kernel with the largest share of the step, at its largest launch (first slab)
        dom = max(("logits", "dH", "dW"), key=lambda st: sum(per[st]))
        rows0 = slabs[1] - slabs[0]
        flops0 = 2.0 * rows0 * spec.d * spec.V
        ach = flops0 / (per[dom][0] * 1e-3) / 1e12
        roofline = {"bound": "tensor", "kernel": STAGE_KERNEL[dom], "launch": f"first row slab ({rows0} rows)",
                    "achieved": ach, "peak": peaks["sustained"], "unit": "TFLOP/s", "frac": ach / peaks["sustained"],
                    "peak_kind": f"{peaks['source']} sustained bf16 (kernel timed inside the step loop); burst {peaks['burst']}",
                    "timed": "CUDA events recorded by cat_loss_fwd_bwd_events around this launch, on the launching stream, in every timed step",
                    "flops_per_launch": flops0, "share_of_step": sum(per[dom]) / ms_per_step,
                    "traffic": TRAFFIC_BYTES.get((f"config{args.config}", T, dom)) if pair else None,
                    "traffic_unit": "bytes per launch (ncu dram__bytes_read.sum + dram__bytes_write.sum)"}
    tflops = value * flops_per_token / 1e12 / world
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if spec.dtype == "bf16" else "f32", "data": "synthetic", "config": cfg,
        "tflops_6TdV_per_gpu": tflops,
        "frac_of_peak": {"measured_burst": tflops / peaks["burst"], "measured_sustained": tflops / peaks["sustained"],
                         "nominal_2250": tflops / 2250.0, "peaks": peaks["source"]},
        "path": "cat_loss_fwd_bwd (softmax numerators kept as bf16 per row slab, 6TdV executed)",
        "two_call_path": {"what": "cat_loss_fwd + cat_loss_bwd (logits recomputed, 8TdV executed)", "ms_per_step": split_ms,
                          "value": world * T / (split_ms * 1e-3), "tflops_6TdV_per_gpu": flops_per_token * T / (split_ms * 1e-3) / 1e12,
                          "fwd_ms": fwd_ms, "bwd_ms": split_ms - fwd_ms},
        "roofline": roofline, "stages": stage_info,
        "roofline_fwd_two_call": {"bound": "tensor", "kernel": "tc::gemm_kernel<K-major,K-major,EpiFwd,pair> (forward logits + online softmax)",
                     "achieved": achieved, "peak": peaks["sustained"], "unit": "TFLOP/s", "frac": achieved / peaks["sustained"],
                     "peak_kind": f"{peaks['source']} sustained bf16 (kernel timed inside the step loop); burst {peaks['burst']}",
                     "timed": "cat_loss_fwd bracketed by CUDA events inside the two-call step loop (GEMM + two O(T) kernels, 0.2 %)",
                     "flops_per_launch": fwd_flops,
                     "traffic": TRAFFIC_BYTES.get((f"config{args.config}", T, "fwd_two_call")) if pair else None,
                     "traffic_unit": "bytes per launch (ncu dram read + write); algorithmic bytes: W + H + partials = %d" % (
                         spec.V * spec.d * 2 + T * spec.d * 2 + 2 * 4 * T * 128)},
        "eq12_path": kd_info,
        "clocks": clocks, "e2e": e2e,
        "gpu_launches": None,
    }
    # launches of our kernels per step of the timed (fused) path, as the library itself counts them:
    # scale + per row slab (logits GEMM, row kernel(s), z->dz, dH GEMM, dW GEMM) + finalize
    per_step = B.cat_loss_launch_count(cl.shape, 2)
    out["gpu_launches"] = per_step * args.steps
    out["launches_per_step"] = per_step

    if not args.no_cpu_baseline:
        rows = 2048            # about 10 s of fp64 work on 16 host cores
        rate, ms = oracle_sample_rate(batch, rows)
        out["cpu_baseline"] = {"value": rate, "unit": UNIT, "cores": host_threads(), "kind": "oracle",
                               "sample": f"first {rows} rows (whole K-blocks) of the workload, fwd+bwd incl. their dW contribution, {ms:.0f} ms"}
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
