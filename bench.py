#!/usr/bin/env python
"""Benchmark of the CAT loss hot path (fused LM head + CAT-weighted cross-entropy, fwd + bwd).

One step = the whole hot path, forward and backward (one cat_loss_fwd_bwd call), over one synthetic
draft-training batch of the Llama-3.2-1B-shaped head config (T=16384 rows in blocks of K=8, d=2048,
V=128256, bf16); the two-call form (cat_loss_fwd + cat_loss_bwd, logits recomputed) is timed beside it.
Prints ONE JSON line.  `value` is tokens/s over exactly --steps steps with inputs resident in HBM;
`sustained` repeats the same step back to back for at least 2 s (the power cap settles the clock only
after a while) with the clocks sampled under it; `e2e` is the same metric with host (pinned) buffers,
host<->device copies inside the timed region; `roofline` is the GEMM with the largest share of the
step, timed by events inside the timed steps, against the measured dense bf16 peak (`stages` has every
stage; `roofline_fwd_two_call` the forward GEMM of the two-call path); `all_configs` times the other
configurations; `cpu_baseline` is the fp64 oracle timed on this machine's host cores on a bounded sample.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 2]

N > 1: one rank per GPU.  Started under torch.distributed.run the ranks are taken from the
environment; started plainly, bench.py starts the N ranks itself (and refuses when fewer than N
devices are visible).  ONE seeded batch of N*T rows is sharded by whole draft blocks (draft blocks are
independent, W replicated): the hot path itself has no data-path collective, weak scaling.  `dp_step`
times what a data-parallel training step adds to it: the all-reduce of dW over NCCL, once after the
one-call path and once slab by slab under the two-call backward.
"""
import argparse
import json
import math
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch

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

    def __init__(self, device_index, period_ms=100):
        self.idx, self.rows, self.proc, self.period = device_index, [], None, period_ms

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", str(self.period), "-i", str(self.idx)], stdout=subprocess.PIPE, text=True)
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
        pw = [float(r[3]) for r in self.rows if len(r) >= 9 and r[3].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = set()
        for r in self.rows:
            if len(r) >= 9:
                for n, v in zip(names, r[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm), power_w_max=max(pw) if pw else None)


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


def visible_devices():
    return torch.cuda.device_count() if torch.cuda.is_available() else 0


def launch_ranks(n, argv):
    """Started plainly with --gpus n > 1: run the n ranks as children, one per device."""
    have = visible_devices()
    if have < n:
        sys.stderr.write(f"bench.py --gpus {n}: {have} CUDA device(s) visible; refusing to report {n} GPUs from fewer\n")
        return 2
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + argv
    return subprocess.call(cmd)


def time_config(cfg_id, dev, local_rank, warmup=3, steps=5):
    """One-call and two-call paths of another configuration: `warmup` + `steps` steps each, clocks sampled."""
    from paper_2605_08632_b200 import synth
    from paper_2605_08632_b200.api import CatLoss
    spec = synth.CONFIGS[cfg_id]
    batch = synth.make_batch(cfg_id)
    H, W = batch.H.to(dev), batch.W.to(dev)
    labels, valid = batch.labels.to(dev), batch.valid.to(dev)
    cl = CatLoss(spec.T, spec.d, spec.V, spec.K, dtype=batch.torch_dtype)
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    peaks = load_peaks()
    out = {"workload": f"config{cfg_id}:{spec.name}", "T": spec.T, "K": spec.K, "d": spec.d, "V": spec.V, "dtype": spec.dtype,
           "steps": steps, "warmup": warmup}

    def one():
        cl.forward_backward(H, W, labels, valid)

    def two():
        cl.forward(H, W, labels, valid)
        cl.backward(H, W, labels, valid)

    for name, fn in (("one_call", one), ("two_call", two)):
        for _ in range(warmup):
            fn()
        torch.cuda.synchronize()
        sampler = ClockSampler(local_rank, period_ms=50)
        sampler.start()
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(steps):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        clocks = sampler.stop()
        ms = e0.elapsed_time(e1) / steps
        tf = 6.0 * spec.T * spec.d * spec.V / (ms * 1e-3) / 1e12
        out[name] = {"ms_per_step": ms, "value": spec.T / (ms * 1e-3), "unit": UNIT, "tflops_6TdV": tf, "clocks": clocks}
        if spec.dtype == "bf16":
            out[name]["frac_of_peak"] = {"measured_burst": tf / peaks["burst"], "measured_sustained": tf / peaks["sustained"]}
    status = cl.fwd_stats().device_status | (cl.fused_status() if spec.dtype == "bf16" else 0) | cl.bwd_status()
    assert status == 0, "device reported a timed-out wait"
    if spec.dtype != "bf16":
        out["note"] = "fp32 FFMA path (fp32 throughout): a correctness configuration, no roofline claim"
    del cl, H, W
    torch.cuda.empty_cache()
    return out


def nccl_summary(log_dir):
    """What NCCL's own log says about the transport (NVLS, rings/trees), from the per-rank debug files."""
    out = {"nvls": False, "files": 0, "log_lines": 0, "lines": []}
    keys = ("NCCL version", "NVLS", "Connected all", "Channel 00", "via P2P", "via SHM", "Using network", "comm 0x")
    try:
        for fn in sorted(os.listdir(log_dir)):
            out["files"] += 1
            with open(os.path.join(log_dir, fn), errors="replace") as f:
                for line in f:
                    out["log_lines"] += 1
                    if "NVLS" in line and "disabled" not in line.lower():
                        out["nvls"] = True
                    if any(k in line for k in keys) and len(out["lines"]) < 10:
                        out["lines"].append(line.strip()[-160:])
    except Exception as e:      # the summary is an extra: never fail the run for it
        out["error"] = repr(e)
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2)
    ap.add_argument("--rows", type=int, default=0, help="override T per GPU (debug / profiling of a small case)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the Eq. 12 timing, the sustained loop and the other configurations")
    ap.add_argument("--profile", choices=["fused", "two-call", "kd"], default=None,
                    help="run only that path for --warmup + --steps steps and exit (for ncu captures of a small case; prints no bench line)")
    args = ap.parse_args()

    env_world = int(os.environ.get("WORLD_SIZE", "0"))
    if args.impl == "ours" and env_world == 0 and args.gpus > 1:
        sys.exit(launch_ranks(args.gpus, sys.argv[1:]))
    rank = int(os.environ.get("RANK", "0"))
    world = max(env_world, 1)
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "ours" and world != args.gpus:
        raise SystemExit(f"bench.py --gpus {args.gpus} was started with WORLD_SIZE={world}: the two must agree")

    from paper_2605_08632_b200 import synth
    spec = synth.CONFIGS[args.config]
    T = args.rows if args.rows else spec.T                       # rows per GPU
    cfg = dict(workload=f"config{args.config}:{spec.name}", T=T * world, K=spec.K, d=spec.d, V=spec.V, rows_per_gpu=T,
               labels=spec.labels, l2="inputs larger than L2 (W alone is %.0f MB)" % (spec.V * spec.d * 2 / 1e6),
               parallelism=f"one seeded batch of {world} x {T} rows sharded by whole draft blocks, W replicated, no collective on the hot path")
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
        cfg["T"] = T
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
    if visible_devices() <= local_rank:
        raise SystemExit(f"bench.py needs CUDA device {local_rank}: there is no CPU path for the product")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    nccl_dir = None
    if env_world >= 1:
        import tempfile
        import torch.distributed as dist
        # NCCL's own log goes to per-rank files (stdout carries the one JSON line); rank 0 summarises them
        nccl_dir = os.environ.get("CAT_BENCH_NCCL_LOG_DIR") or tempfile.mkdtemp(prefix="cat_bench_nccl_")
        os.environ.setdefault("NCCL_DEBUG", "INFO")
        os.environ.setdefault("NCCL_DEBUG_SUBSYS", "INIT,ENV")
        os.environ.setdefault("NCCL_DEBUG_FILE", os.path.join(nccl_dir, "rank%h_%p.log"))
        dist.init_process_group("nccl", device_id=dev)
    from paper_2605_08632_b200.api import CatLoss
    from paper_2605_08632_b200 import binding as B
    from paper_2605_08632_b200 import ncu_traffic
    from paper_2605_08632_b200.data_parallel import CudaEngine, DataParallelCatLoss, shard_rows

    # one seeded batch of world * T rows; this rank takes its whole-block share of it
    whole = synth.make_batch(args.config, T=T * world)
    r0, r1 = shard_rows(T * world, spec.K, world, rank)
    assert r1 - r0 == T
    batch = synth.Batch(whole.spec, T, whole.K, whole.d, whole.V, whole.H[r0:r1].contiguous(), whole.W, whole.labels[r0:r1].contiguous(),
                        whole.valid[r0:r1].contiguous(), whole.biased[r0:r1].contiguous())
    del whole
    H, W = batch.H.to(dev), batch.W.to(dev)
    labels, valid = batch.labels.to(dev), batch.valid.to(dev)
    cl = CatLoss(T, spec.d, spec.V, spec.K, dtype=batch.torch_dtype)

    def step():
        cl.forward_backward(H, W, labels, valid)

    def step_split():
        cl.forward(H, W, labels, valid)
        cl.backward(H, W, labels, valid)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def reduce_max(ms):
        if dist is not None:
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
        print(json.dumps({"profile_run": args.profile, "T": T, "source_digest": ncu_traffic.source_digest(), "note": "not a benchmark value"}))
        return

    stream = torch.cuda.current_stream()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    warmup = max(args.warmup, 3)

    # ---- headline: the fused call (cat_loss_fwd_bwd: logits kept per row slab, 6*T*d*V executed)
    for _ in range(warmup):
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

    # ---- the same step back to back for at least 2 s: the clock the power cap settles at, and time x clock
    sustained = None
    if not args.no_extras:
        n_sus = max(args.steps, int(math.ceil(2000.0 / ms_per_step)))
        barrier()
        sampler = ClockSampler(local_rank)
        sampler.start()
        barrier()
        ev0.record(stream)
        for _ in range(n_sus):
            step()
        ev1.record(stream)
        barrier()
        sus_clocks = sampler.stop()
        sus_ms = reduce_max(ev0.elapsed_time(ev1)) / n_sus
        sustained = {"steps": n_sus, "ms_per_step": sus_ms, "value": world * T / (sus_ms * 1e-3), "unit": UNIT,
                     "tflops_6TdV_per_gpu": flops_per_token * T / (sus_ms * 1e-3) / 1e12, "clocks": sus_clocks,
                     "ms_x_sm_mhz": sus_ms * sus_clocks["sm_mhz"] if sus_clocks.get("sm_mhz") else None}

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

    # ---- data-parallel training step: the hot path plus the all-reduce of dW (and of N and the loss sums)
    dp_info = None
    if dist is not None and spec.dtype == "bf16":
        dp_info = {"what": "DataParallelCatLoss.step over NCCL: global N, local loss + gradients scaled by g/N_global, all-reduce of dW "
                           "(%.2f GB fp32) and of the loss sums" % (spec.V * spec.d * 4 / 1e9), "world": world}
        dp_steps = max(3, min(args.steps, 10))
        for name, overlap in (("one_call_then_allreduce", False), ("two_call_slabwise_overlap", True)):
            eng = CudaEngine(T, spec.d, spec.V, spec.K, dtype=batch.torch_dtype)
            dp = DataParallelCatLoss(eng, overlap=overlap)
            for _ in range(3):
                dp.step(H, W, labels, valid)
            barrier()
            ev0.record(stream)
            for _ in range(dp_steps):
                dp.step(H, W, labels, valid)
            ev1.record(stream)
            barrier()
            ms = reduce_max(ev0.elapsed_time(ev1)) / dp_steps
            dp_info[name] = {"ms_per_step": ms, "value": world * T / (ms * 1e-3), "unit": UNIT, "steps": dp_steps}
            del dp, eng
            torch.cuda.empty_cache()

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
        del cls, ins, Hh, Wh, dH_h, dW_h
        torch.cuda.empty_cache()

    if rank != 0:
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    fwd_flops = 2.0 * T * spec.d * spec.V
    achieved = fwd_flops / (fwd_ms * 1e-3) / 1e12
    pair = os.environ.get("CAT_LOSS_CTA_PAIR", "1") != "0"
    # DRAM bytes per launch from the recorded ncu capture of this workload; None when there is none for it
    # or the kernel sources changed since (see paper_2605_08632_b200/ncu_traffic.py)
    workload_key = f"config{args.config}"
    traffic_fused = ncu_traffic.load(workload_key, T, "fused") if pair else None
    traffic_two = ncu_traffic.load(workload_key, T, "two-call") if pair else None

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
        if traffic_fused:
            stage_info["dram_bytes_per_launch"] = {st: [ncu_traffic.bytes_of(traffic_fused, st, sl, n_slabs) for sl in range(n_slabs)]
                                                   for st in ("logits", "dH", "dW")}
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
                    "traffic": ncu_traffic.bytes_of(traffic_fused, dom, 0, n_slabs),
                    "traffic_unit": "bytes per launch (ncu dram__bytes_read.sum + dram__bytes_write.sum of the recorded capture; "
                                    "null when the kernel sources changed since)"}
    tflops = value * flops_per_token / 1e12 / world
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if spec.dtype == "bf16" else "f32", "data": "synthetic", "config": cfg,
        "tflops_6TdV_per_gpu": tflops,
        "frac_of_peak": {"measured_burst": tflops / peaks["burst"], "measured_sustained": tflops / peaks["sustained"],
                         "nominal_2250": tflops / 2250.0, "peaks": peaks["source"]},
        "path": "cat_loss_fwd_bwd (softmax numerators kept as bf16 per row slab, 6TdV executed)",
        "sustained": sustained,
        "two_call_path": {"what": "cat_loss_fwd + cat_loss_bwd (logits recomputed, 8TdV executed)", "ms_per_step": split_ms,
                          "value": world * T / (split_ms * 1e-3), "tflops_6TdV_per_gpu": flops_per_token * T / (split_ms * 1e-3) / 1e12,
                          "fwd_ms": fwd_ms, "bwd_ms": split_ms - fwd_ms},
        "roofline": roofline, "stages": stage_info,
        "roofline_fwd_two_call": {"bound": "tensor", "kernel": "tc::gemm_kernel<K-major,K-major,EpiFwd,pair> (forward logits + online softmax)",
                     "achieved": achieved, "peak": peaks["sustained"], "unit": "TFLOP/s", "frac": achieved / peaks["sustained"],
                     "peak_kind": f"{peaks['source']} sustained bf16 (kernel timed inside the step loop); burst {peaks['burst']}",
                     "timed": "cat_loss_fwd bracketed by CUDA events inside the two-call step loop (GEMM + two O(T) kernels, 0.2 %)",
                     "flops_per_launch": fwd_flops,
                     "traffic": ncu_traffic.bytes_of(traffic_two, "fwd_two_call", 0, 1),
                     "traffic_unit": "bytes per launch (ncu dram read + write); algorithmic bytes: W + H + partials = %d" % (
                         spec.V * spec.d * 2 + T * spec.d * 2 + 2 * 4 * T * 128)},
        "eq12_path": kd_info, "dp_step": dp_info,
        "clocks": clocks, "e2e": e2e,
        "gpu_launches": None,
    }
    # launches of our kernels per step of the timed (fused) path, as the library itself counts them:
    # scale + per row slab (logits GEMM, row kernel(s), z->dz, dH GEMM, dW GEMM) + finalize
    per_step = B.cat_loss_launch_count(cl.shape, 2)
    out["gpu_launches"] = per_step * args.steps * world
    out["launches_per_step"] = per_step
    table, n_first = B.cat_die_map()
    out["die_map"] = {"tpcs": len(table), "tpcs_on_first_die": n_first,
                      "what": "SM-to-die table measured by the library on this device; the GEMM kernels number their CTA pairs by it (0 tpcs: not usable, blockIdx order)"}
    if dist is not None:
        out["nccl"] = nccl_summary(nccl_dir)

    # ---- the other configurations (one GPU): config 1's time, configs 3, 4, 5 on both paths
    if not args.no_extras and world == 1:
        del cl, H, W
        torch.cuda.empty_cache()
        out["all_configs"] = [time_config(c, dev, local_rank, steps=20 if c == 1 else 5) for c in (1, 3, 4, 5) if c != args.config]

    if not args.no_cpu_baseline and world == 1:
        rows = 2048            # about 10 s of fp64 work on 16 host cores
        rate, ms = oracle_sample_rate(batch, rows)
        out["cpu_baseline"] = {"value": rate, "unit": UNIT, "cores": host_threads(), "kind": "oracle",
                               "sample": f"first {rows} rows (whole K-blocks) of the workload, fwd+bwd incl. their dW contribution, {ms:.0f} ms"}
    print(json.dumps(out))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
