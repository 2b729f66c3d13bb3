#!/usr/bin/env python
"""Benchmark of the DP-SGD privatised-gradient step at BERT-Large shapes.

One step = one microbatch of 256 examples x 128 tokens through the whole path on one GPU:
per-example norms over 24 encoder blocks + the token embedding -> clip factors -> clipped accumulate
-> fused noise + scaling + AdamW over ~334M fp32 parameters.  Inputs are seeded and synthetic and
stay resident in HBM (32 GB per microbatch, far larger than L2, so no flush is needed).

  python bench.py [--gpus N] [--steps K] [--warmup W]          device-timed line (+ e2e, roofline, cpu_baseline)
  python bench.py --impl reference ...                         the CPU checker timed on the host cores
  python bench.py --macro-microbatches 8192                    one whole macro-step of the 2,097,152-example mega-batch
  python bench.py --long-sequence-paths                        T=512 block: Gram vs materialised vs auto-selected norms

Under torchrun (N > 1) each rank processes its own microbatches (weak scaling); the accumulators are
reduce-scattered once per step, the noise/AdamW pass runs on the local shard and theta is all-gathered.
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
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of one k_accum_pair launch over TWO encoder blocks
# (`--blocks 2`, 2.7 GB on the device), from an `ncu --set full` capture of that small case.
# The kernel's traffic grows with the number of blocks (every block's operands are read once, its accumulators read
# and written once), so a launch over n blocks is reported as this figure x n / 2.  Not to be re-taken on the full
# 32 GB workload.  Set to None whenever that kernel changes until the capture has been repeated.
ACCUM_TRAFFIC_2BLOCKS_BYTES = 2.436e9
HBM_NOMINAL_GBS = 8000.0          # the figure the target quotes; fractions are reported against it and the measured copy

METRIC = "dp_sgd_examples_per_s_bert_large"
UNIT = "examples/s"
WORKLOAD = "bert_large"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "tf_burst": p["bf16_tflops"], "tf_sustained": p["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "tf_burst": 1590.0, "tf_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.rows = []
        self.proc = None
        try:
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            self.cmd = ["nvidia-smi", f"--id={uuid}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                        "-lms", "100"]
        except Exception:
            self.cmd = None

    def start(self):
        if self.cmd is None:
            return
        try:
            self.proc = subprocess.Popen(self.cmd, stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            f = [x.strip() for x in r.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
                pw.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm), "power_w": float(np.mean(pw)) if pw else None}


def config_dict(wl, n_params, n_gpus, blocks=24):
    """The workload description, identical in both arms."""
    return {"workload": WORKLOAD if blocks == 24 else f"{WORKLOAD}[first {blocks} blocks only]",
            "B": wl.B, "T": wl.T, "layers": len(wl.specs), "params": n_params, "microbatches_per_step": 1,
            "parallelism": f"dp{n_gpus}", "l2": "inputs (32 GB per microbatch) far exceed L2; no flush"}


def oracle_layers(data, rows):
    from oracle import dp_oracle as O
    out = []
    for ld in data:
        out.append(O.OracleLayer(kind=ld.spec.kind, G=ld.G[rows].double().cpu().numpy(),
                                 A=None if ld.A is None else ld.A[rows].double().cpu().numpy(),
                                 ids=None if ld.ids is None else ld.ids[rows].cpu().numpy().astype(np.int64),
                                 has_bias=ld.spec.has_bias, vocab=ld.spec.d_in if ld.spec.kind == "embedding" else 0))
    return out


def oracle_threads() -> int:
    """Threads the checker's numpy calls can use: the size of numpy's BLAS pool (its matrix products are the only
    multi-threaded part), bounded by the cores this process may run on."""
    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    try:
        from threadpoolctl import threadpool_info
        pools = [p["num_threads"] for p in threadpool_info() if p.get("user_api") == "blas"
                 and "numpy" in (p.get("filepath") or "")]
        return min(cores, max(pools)) if pools else cores
    except Exception:
        return cores


def time_oracle(wl, data, n_params, budget_s=15.0, max_examples=8, threads=None):
    """The CPU checker as it stands on a bounded sample: k examples through every layer (norms, clip,
    accumulate) plus noise + AdamW on 1/64 of the parameters; scaled linearly to one 256-example step.
    threads: cap on numpy's BLAS pool for this measurement (None: as the process found it)."""
    if threads is not None:
        from threadpoolctl import threadpool_limits
        with threadpool_limits(limits=threads, user_api="blas"):
            out = time_oracle(wl, data, n_params, budget_s, max_examples)
        out["cores"] = threads
        return out
    from oracle import dp_oracle as O
    t0 = time.perf_counter()
    k = 0
    accs = None
    while k < max_examples:
        ol = oracle_layers(data, slice(k, k + 1))
        ta = time.perf_counter()
        n = O.per_example_sqnorms(ol)
        c = O.clip_factors(n, wl.C)
        accs = O.zero_accumulators(ol) if accs is None else accs
        O.clipped_accumulate(ol, c, accs)
        per_ex = time.perf_counter() - ta
        k += 1
        if time.perf_counter() - t0 + per_ex > budget_s:
            break
    t_examples = time.perf_counter() - t0
    # time only the arithmetic, not the device->host conversion of inputs
    frac = 64
    n_s = n_params // frac
    S = np.zeros(n_s)
    th = np.zeros(n_s)
    tb = time.perf_counter()
    g = O.add_noise_and_scale(S, wl.sigma, wl.C, wl.B, 0, 1, 0)
    O.adamw_step(th, th, th, g, wl.lr, wl.beta1, wl.beta2, wl.xi, wl.weight_decay, 1)
    t_update = (time.perf_counter() - tb) * frac
    step_s = t_examples / k * wl.B + t_update
    return {"value": wl.B / step_s, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
            "sample": f"{k} of {wl.B} examples through all {len(data)} layers (incl. host conversion of their "
                      f"inputs) + noise/AdamW on 1/{frac} of {n_params} parameters, scaled linearly to one step "
                      f"(extrapolated); measured {t_examples:.1f}s + {t_update / frac:.1f}s"}


def run_reference(args):
    """The reference arm: the CPU checker (numpy, fp64) on the host cores, same config and metric."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2108_01624_b200 import synth
    wl = synth.workload(WORKLOAD)
    n_params = wl.n_params()
    data = synth.generate(wl, seed=0, device="cpu", B=4)
    values = []
    cb = None
    for it in range(args.warmup + args.steps):
        budget = 3.0 if it < args.warmup else max(4.0, 60.0 / max(1, args.steps))
        cb = time_oracle(wl, data, n_params, budget_s=budget, max_examples=4)
        if it >= args.warmup:
            values.append(cb["value"])
    v = float(np.mean(values)) if values else cb["value"]
    cb["value"] = v
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * wl.B / v, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(wl, n_params, args.gpus),
            "cpu_baseline": cb,
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the per-phase power loops and the other workloads' timings (profiler captures)")
    ap.add_argument("--fused-reduce", action="store_true",
                    help="N > 1: end each step with ONE kernel per rank over the ranks' peer-mapped accumulators and "
                         "replicas (dp_reduce_noise_adamw_step) instead of reduce-scatter + update + all-gather")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--blocks", type=int, default=24,
                    help="encoder blocks of the stack (24 = the benchmark workload; fewer only for profiler captures)")
    ap.add_argument("--macro-microbatches", type=int, default=0,
                    help="instead of the per-microbatch line: time ONE macro-step of this many microbatches "
                         "(8192 = the 2,097,152-example mega-batch of Section 5.3) and print its line")
    ap.add_argument("--long-sequence-paths", action="store_true",
                    help="instead of the per-microbatch line: the T=512 BERT-Large block (B=64) with the norm path of "
                         "its linear layers forced to Gram, forced to materialised tiles, and chosen automatically")
    ap.add_argument("--verify", action="store_true",
                    help="with --macro-microbatches: check the accumulator after the loop (untimed) against the "
                         "counted sum of single passes over the pool, and against the bound N C")
    ap.add_argument("--pool", type=int, default=2,
                    help="distinct resident microbatches the macro-step rotates over (32 GB each)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    args.warmup = max(args.warmup, 3)
    if args.long_sequence_paths:
        run_long_sequence_paths(args)
        return

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    # One rank per GPU.  With fewer GPUs than ranks (a functional check of the N > 1 path on one GPU; no kernel of
    # this library waits for another rank) the ranks share devices, and DP_BENCH_BACKEND=gloo replaces NCCL, which
    # refuses two ranks on one device.
    local = local % max(1, torch.cuda.device_count())
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        backend = os.environ.get("DP_BENCH_BACKEND", "nccl")
        if backend == "nccl":
            dist.init_process_group("nccl", device_id=dev)
        else:
            dist.init_process_group(backend)

    import paper_2108_01624_b200 as pkg
    from paper_2108_01624_b200 import build as builder
    from paper_2108_01624_b200 import synth
    from paper_2108_01624_b200.parallel import ShardedUpdate
    if rank == 0:
        builder.build()
    if dist is not None:
        dist.barrier()

    wl = synth.workload(WORKLOAD)
    if args.blocks != 24:
        wl.specs = wl.specs[:6 * args.blocks] + [wl.specs[-1]]
    data = synth.generate(wl, seed=1000 + rank, device=dev)
    step = pkg.DPStep(wl.specs, dev, wl.C, wl.sigma, wl.lr, wl.beta1, wl.beta2, wl.xi, wl.weight_decay, seed=0,
                      shard_world=world)
    step.theta.copy_(synth.initial_weights(step.n_flat, 0, dev))
    n_params = wl.n_params()
    lin_idx = [k for k, sp in enumerate(wl.specs) if sp.kind == "linear"]
    rest_idx = [k for k, sp in enumerate(wl.specs) if sp.kind != "linear"]
    ll_all = step.layer_list(data)
    ll_lin = pkg.LayerList([ll_all.layers[k] for k in lin_idx])
    ll_rest = pkg.LayerList([ll_all.layers[k] for k in rest_idx])
    # The model is passed in two calls (linear layers; LayerNorm + embedding) so that the accumulate GEMM can be
    # bracketed by events of its own; each list has its workspace, and the second accumulate reuses the
    # LayerNorm column sums its norm call left there.
    ws = torch.empty(max(pkg.dp_workspace_bytes(ll_lin), 256), dtype=torch.uint8, device=dev)
    ws_rest = torch.empty(max(pkg.dp_workspace_bytes(ll_rest), 256), dtype=torch.uint8, device=dev)
    sq = torch.empty(wl.B, dtype=torch.float32, device=dev)
    clip = torch.empty(wl.B, dtype=torch.float32, device=dev)
    sharded = None
    if world > 1 and args.fused_reduce:
        # every rank's accumulator and replica of theta mapped into this process (CUDA IPC; plain loads and stores)
        from paper_2108_01624_b200.parallel import exchange_peer_buffers
        peers = (exchange_peer_buffers(step.acc, dist, world, rank), exchange_peer_buffers(step.theta, dist, world, rank))
        sharded = ShardedUpdate(step, dist, world, rank, peer_acc=peers[0], peer_theta=peers[1])
    elif world > 1:
        sharded = ShardedUpdate(step, dist, world, rank)
    if sharded is not None:
        sharded.time_phases()
    stream = torch.cuda.current_stream()

    if args.macro_microbatches > 0:
        run_macro_step(args, pkg, synth, wl, step, sharded, dist, world, rank, dev, data, lin_idx, rest_idx,
                       (ws, ws_rest, sq, clip), stream)
        if dist is not None:
            dist.destroy_process_group()
        return

    def make_lists(d):
        ll = step.layer_list(d)
        return pkg.LayerList([ll.layers[k] for k in lin_idx]), pkg.LayerList([ll.layers[k] for k in rest_idx])

    def one_step(ev=None, lists=None):
        lin, rest = (ll_lin, ll_rest) if lists is None else lists
        if ev:
            ev[0].record(stream)
        pkg.dp_per_example_sqnorms(lin, sq, False, ws)
        pkg.dp_per_example_sqnorms(rest, sq, True, ws_rest)
        pkg.dp_clip_factors(sq, wl.C, clip)
        if ev:
            ev[1].record(stream)
        pkg.dp_clipped_accumulate(lin, clip, ws)
        if ev:
            ev[2].record(stream)
        pkg.dp_clipped_accumulate_after_sqnorms(rest, clip, ws_rest)
        if ev:
            ev[3].record(stream)
        step.examples_seen = wl.B * world
        # the status word is read once after the loop, not with a host synchronisation in every step
        if sharded is None:
            step.finish_macro_batch(check_status=False)
        else:
            sharded.finish_macro_batch(check_status=False)
        if ev:
            ev[4].record(stream)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        one_step()
    barrier()
    if pkg.dp_poll_status() != 0:
        raise RuntimeError("device status not clean after warm-up")

    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(args.steps)]
    if sharded is not None:
        sharded.timings()          # drop the warm-up steps' records
    sampler = ClockSampler(local)
    sampler.start()
    l0 = pkg.dp_launch_count()
    barrier()
    t_start = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    t_start.record(stream)
    for k in range(args.steps):
        one_step(evs[k])
    t_end.record(stream)
    barrier()
    launches = pkg.dp_launch_count() - l0
    clocks = sampler.stop()
    if pkg.dp_poll_status() != 0:
        raise RuntimeError("device status not clean after the timed steps")
    total_ms = t_start.elapsed_time(t_end)
    if dist is not None:
        t = torch.tensor([total_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    ms_per_step = total_ms / args.steps
    value = wl.B * world / (ms_per_step * 1e-3)
    phases = np.array([[e[i].elapsed_time(e[i + 1]) for i in range(4)] for e in evs]).mean(axis=0)
    # N > 1: the exchange inside the last phase (reduce-scatter | update | all-gather, or barrier | fused kernel |
    # barrier), device milliseconds on this rank, mean over the timed steps
    collective = sharded.timings() if sharded is not None else None
    if collective is not None:
        collective["way"] = "one kernel over peer memory" if args.fused_reduce else "reduce-scatter + all-gather, in place"

    peaks = measured_peaks()
    T, B = wl.T, wl.B
    flops_acc = sum(2.0 * B * T * wl.specs[k].d_in * wl.specs[k].d_out for k in lin_idx)
    ach_tf = flops_acc / (phases[1] * 1e-3) / 1e12
    bytes_acc = sum(2.0 * B * T * (wl.specs[k].d_in + wl.specs[k].d_out)
                    + 8.0 * wl.specs[k].d_in * wl.specs[k].d_out for k in lin_idx)
    traffic = None if ACCUM_TRAFFIC_2BLOCKS_BYTES is None else ACCUM_TRAFFIC_2BLOCKS_BYTES * args.blocks / 2.0
    roofline = {"kernel": "clipped-accumulate GEMM (all linear layers, one call)", "bound": "tensor",
                "achieved": ach_tf, "peak": peaks["tf_sustained"], "unit": "TFLOP/s",
                "frac": ach_tf / peaks["tf_sustained"], "frac_of_burst": ach_tf / peaks["tf_burst"],
                "peak_source": peaks["source"] + " (sustained bf16; kernel timed inside a long step)",
                "traffic": traffic, "traffic_source": "ncu capture of a 2-block launch, scaled by blocks / 2",
                "algorithmic_bytes": bytes_acc}
    bytes_norm = sum(2.0 * B * T * (wl.specs[k].d_in + wl.specs[k].d_out) for k in lin_idx) \
        + sum(2.0 * 2 * B * T * wl.specs[k].d_out for k in rest_idx if wl.specs[k].kind == "layernorm") \
        + sum(2.0 * B * T * wl.specs[k].d_out + 4.0 * B * T for k in rest_idx if wl.specs[k].kind == "embedding")
    bytes_upd = 32.0 * step.n_flat
    # algorithmic flops of the Gram norms: the upper triangle (with the diagonal) of each T x T Gram, i.e. half of
    # 2 T^2 (d_in + d_out) up to the diagonal -- whatever the kernel executes
    flops_gram = sum(2.0 * B * (T * (T + 1) / 2.0) * (wl.specs[k].d_in + wl.specs[k].d_out) for k in lin_idx)
    tf_both = (flops_acc + flops_gram) / ((phases[0] + phases[1]) * 1e-3) / 1e12

    def hbm(nbytes, ms):
        gbs = nbytes / (ms * 1e-3) / 1e9
        return {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": gbs / peaks["hbm_gbs"], "frac_of_nominal_8TBs": gbs / HBM_NOMINAL_GBS}
    extra = {
        "norm_pass": hbm(bytes_norm, phases[0]),
        "noise_adamw": hbm(bytes_upd, phases[3]),
        "gram_plus_accumulate": {"bound": "tensor", "achieved": tf_both, "unit": "TFLOP/s",
                                 "algorithmic_flops": flops_acc + flops_gram,
                                 "frac_of_sustained": tf_both / peaks["tf_sustained"],
                                 "frac_of_burst": tf_both / peaks["tf_burst"],
                                 "note": "flop-weighted over the norm pass and the accumulate GEMM; the norm pass is "
                                         "bound by HBM (intensity T = 128 flop/B), so its time counts in full"},
    }

    others = None
    energy = None
    if world == 1 and not args.no_extras:
        energy = phase_energy(pkg, wl, local, stream, step,
                              {"norms+clip": lambda: (pkg.dp_per_example_sqnorms(ll_lin, sq, False, ws),
                                                      pkg.dp_per_example_sqnorms(ll_rest, sq, True, ws_rest),
                                                      pkg.dp_clip_factors(sq, wl.C, clip)),
                               "accumulate_linear": lambda: pkg.dp_clipped_accumulate(ll_lin, clip, ws),
                               "noise_adamw": lambda: step.finish_macro_batch(batch_size=wl.B, check_status=False)},
                              {"norms+clip": phases[0], "accumulate_linear": phases[1], "noise_adamw": phases[3]})
        others = {"megabatch_proxy": megabatch_proxy(pkg, synth, wl, step, data, lin_idx, rest_idx,
                                                     (ws, ws_rest, sq, clip), stream, rank, dev, n_micro=64)}
    e2e = None
    if not args.no_e2e and world == 1:
        e2e = run_e2e(pkg, synth, wl, data, one_step, make_lists, clip, stream, args.e2e_steps)
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline = time_oracle(wl, data, n_params)
        one = time_oracle(wl, data, n_params, budget_s=1.0, max_examples=1, threads=1)
        cpu_baseline["single_thread"] = {"value": one["value"], "unit": UNIT, "cores": 1, "sample": one["sample"]}
    if others is not None:
        # the other workloads, after the 32 GB stack has been released
        del data, ll_all, ll_lin, ll_rest, ws, ws_rest, step, sharded
        torch.cuda.empty_cache()
        others["bert_base_layer"] = small_workload(pkg, synth, "bert_base_layer", dev, stream, reps=50)
        others["bert_large_layer_t512"] = long_sequence_paths(pkg, synth, dev, stream, args.warmup, max(args.steps, 10))

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": config_dict(wl, n_params, world, args.blocks),
                "phases_ms": {"norms+clip": phases[0], "accumulate_linear": phases[1],
                              "accumulate_ln_embedding": phases[2], "noise_adamw": phases[3]},
                "collective_ms": collective, "roofline": roofline, "rooflines_other": extra,
                "phase_energy": energy, "other_workloads": others, "cpu_baseline": cpu_baseline, "e2e": e2e,
                "gpu_launches": int(launches), "clocks": clocks}
        print(json.dumps(line))
    if dist is not None:
        if args.fused_reduce:          # unmap the peers' buffers before any owner exits
            barrier()
            sharded = peers = None
            torch.cuda.ipc_collect()
            barrier()
        dist.destroy_process_group()


def phase_energy(pkg, wl, device_index, stream, step, fns, in_step_ms, seconds=3.0):
    """Each phase of the step repeated ALONE, back to back, for about `seconds`, with the clock and power sampler
    running (samples of the first 1.2 s dropped): its time per repetition, the mean board power and the median SM clock while it ran, and the energy of
    one repetition (power x time).  Beside it the phase's time inside the step, where the phases alternate every
    few milliseconds under one power cap."""
    out = {}
    for name, fn in fns.items():
        reps = max(3, int(seconds * 1e3 / max(in_step_ms[name], 1e-3)))
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        sampler = ClockSampler(device_index)
        sampler.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        t_host = time.perf_counter()
        n_settled = None
        for _ in range(reps):
            fn()
            if n_settled is None and time.perf_counter() - t_host > 1.2:
                stream.synchronize()           # the launches run ahead of the device: meet it once, then count samples
                n_settled = len(sampler.rows)
        e1.record(stream)
        torch.cuda.synchronize()
        # the power reading is a moving average: only samples taken after more than a second under load count
        sampler.rows = sampler.rows[(n_settled if n_settled is not None else 0) + 1:]
        c = sampler.stop()
        ms = e0.elapsed_time(e1) / reps
        out[name] = {"ms_alone": ms, "ms_in_step": in_step_ms[name], "repetitions": reps, "power_w": c["power_w"],
                     "sm_mhz": c["sm_mhz"], "reasons": c["reasons"], "samples": c["samples"],
                     "joules": None if c["power_w"] is None else c["power_w"] * ms * 1e-3}
    if pkg.dp_poll_status() != 0:
        raise RuntimeError("device status not clean after the per-phase loops")
    return out


def megabatch_proxy(pkg, synth, wl, step, data0, lin_idx, rest_idx, bufs, stream, rank, dev, n_micro):
    """A short stand-in for the 8192-microbatch macro-step (`--macro-microbatches 8192` runs the real one): n_micro
    microbatches rotating over two distinct resident inputs, accumulated in place, then one noise + AdamW pass."""
    ws, ws_rest, sq, clip = bufs
    second = synth.generate(wl, seed=1000 + rank, device=dev, microbatch=1)
    lists = []
    for d in (data0, second):
        ll = step.layer_list(d)
        lists.append((pkg.LayerList([ll.layers[k] for k in lin_idx]), pkg.LayerList([ll.layers[k] for k in rest_idx])))

    def microbatch(k):
        lin, rest = lists[k % 2]
        pkg.dp_per_example_sqnorms(lin, sq, False, ws)
        pkg.dp_per_example_sqnorms(rest, sq, True, ws_rest)
        pkg.dp_clip_factors(sq, wl.C, clip)
        pkg.dp_clipped_accumulate(lin, clip, ws)
        pkg.dp_clipped_accumulate_after_sqnorms(rest, clip, ws_rest)

    step.discard_macro_batch()
    for k in range(3):
        microbatch(k)
    step.discard_macro_batch()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for k in range(n_micro):
        microbatch(k)
    step.examples_seen = wl.B * n_micro
    step.finish_macro_batch(check_status=False)
    e1.record(stream)
    torch.cuda.synchronize()
    if pkg.dp_poll_status() != 0:
        raise RuntimeError("device status not clean after the mega-batch proxy")
    ms = e0.elapsed_time(e1)
    del lists, second
    torch.cuda.empty_cache()
    return {"workload": f"bert_large x {n_micro} microbatches, then one noise + AdamW pass (stand-in for the "
                        "8192-microbatch mega-batch)", "microbatches": n_micro, "examples": wl.B * n_micro,
            "ms": ms, "ms_per_microbatch": ms / n_micro, "examples_per_s": wl.B * n_micro / (ms * 1e-3)}


def small_workload(pkg, synth, name, dev, stream, reps):
    """One of the smaller workloads through the same calls: per-phase device times over `reps` repetitions."""
    wl = synth.workload(name)
    data = synth.generate(wl, seed=0, device=dev)
    step = pkg.DPStep(wl.specs, dev, wl.C, wl.sigma, wl.lr, wl.beta1, wl.beta2, wl.xi, wl.weight_decay, seed=0)
    ll = step.layer_list(data)
    ws = pkg.alloc_workspace(ll)
    sq = torch.empty(wl.B, dtype=torch.float32, device=dev)
    clip = torch.empty_like(sq)
    flush = torch.empty(96 * 1024 * 1024, dtype=torch.float32, device=dev)     # 384 MB > L2, written between repetitions

    def one(ev=None):
        flush.fill_(0.0)
        if ev:
            ev[0].record(stream)
        pkg.dp_per_example_sqnorms(ll, sq, False, ws)
        pkg.dp_clip_factors(sq, wl.C, clip)
        if ev:
            ev[1].record(stream)
        pkg.dp_clipped_accumulate_after_sqnorms(ll, clip, ws)
        if ev:
            ev[2].record(stream)
        step.examples_seen = wl.B
        step.finish_macro_batch(check_status=False)
        if ev:
            ev[3].record(stream)

    for _ in range(3):
        one()
    torch.cuda.synchronize()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(reps)]
    for k in range(reps):
        one(evs[k])
    torch.cuda.synchronize()
    if pkg.dp_poll_status() != 0:
        raise RuntimeError("device status not clean")
    ph = np.array([[e[i].elapsed_time(e[i + 1]) for i in range(3)] for e in evs]).mean(axis=0)
    lin = [sp for sp in wl.specs if sp.kind == "linear"]
    flops = sum(2.0 * wl.B * wl.T * sp.d_in * sp.d_out for sp in lin)
    nbytes = sum(2.0 * wl.B * wl.T * (sp.d_in + sp.d_out) for sp in lin) \
        + sum(4.0 * wl.B * wl.T * sp.d_out for sp in wl.specs if sp.kind == "layernorm")
    total = float(ph.sum())
    return {"workload": name, "B": wl.B, "T": wl.T, "params": wl.n_params(), "repetitions": reps,
            "l2": "384 MB written between repetitions",
            "ms": total, "examples_per_s": wl.B / (total * 1e-3),
            "phases_ms": {"norms+clip": ph[0], "accumulate": ph[1], "noise_adamw": ph[2]},
            "norms_GBs": nbytes / (ph[0] * 1e-3) / 1e9, "accumulate_TFLOPs": flops / (ph[1] * 1e-3) / 1e12}


def long_sequence_paths(pkg, synth, dev, stream, warmup, reps):
    """The long-sequence crossover: one BERT-Large block at T=512, B=64.  Norms of the four linear layers with the
    path forced per layer (token Gram / materialised tiles) and auto-selected, then the clipped accumulate; each
    call device-timed alone over `reps` repetitions (inputs 1.07 GB, larger than L2)."""
    from paper_2108_01624_b200 import binding as b
    wl = synth.workload("bert_large_layer_t512")
    data = [ld for ld in synth.generate(wl, seed=0, device=dev) if ld.spec.kind == "linear"]
    accs = [(torch.zeros(ld.spec.d_in, ld.spec.d_out, device=dev), torch.zeros(ld.spec.d_out, device=dev)) for ld in data]
    sq = torch.empty(wl.B, dtype=torch.float32, device=dev)
    clip = torch.empty_like(sq)

    def timed(fn):
        for _ in range(warmup):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    T, B = wl.T, wl.B
    nbytes = sum(2.0 * B * T * (ld.spec.d_in + ld.spec.d_out) for ld in data)
    nblk = (T + 127) // 128
    flops = {"gram": sum(2.0 * B * (ld.spec.d_in + ld.spec.d_out) * 128 * 128 * nblk * (nblk + 1) / 2 for ld in data),
             "materialized": sum(2.0 * B * T * ld.spec.d_in * ld.spec.d_out for ld in data)}
    out = {}
    l0 = pkg.dp_launch_count()
    for name, path in (("gram", b.DP_PATH_GRAM), ("materialized", b.DP_PATH_MATERIALIZED), ("auto", b.DP_PATH_AUTO)):
        ll = pkg.LayerList([b.Layer(kind="linear", G=ld.G, A=ld.A, acc_w=a[0], acc_b=a[1], has_bias=True, path=path)
                            for ld, a in zip(data, accs)])
        ws = b.alloc_workspace(ll)
        ms = timed(lambda: pkg.dp_per_example_sqnorms(ll, sq, False, ws))
        out[name] = {"ms": ms, "GB/s": nbytes / ms / 1e6}
        if name in flops:       # flops the kernel executes (upper-triangle block pairs for the Gram path)
            out[name]["TFLOP/s"] = flops[name] / ms / 1e9
    pkg.dp_clip_factors(sq, wl.C, clip)
    ms = timed(lambda: pkg.dp_clipped_accumulate(ll, clip, ws))
    out["accumulate"] = {"ms": ms, "TFLOP/s": flops["materialized"] / ms / 1e9}
    torch.cuda.synchronize()
    if pkg.dp_poll_status() != 0:
        raise RuntimeError("device status not clean")
    return {"workload": "bert_large_layer_t512", "B": B, "T": T, "linear_layers": len(data),
            "input_bytes": nbytes, "repetitions": reps, "timings": out,
            "gpu_launches": int(pkg.dp_launch_count() - l0)}


def run_long_sequence_paths(args):
    import paper_2108_01624_b200 as pkg
    from paper_2108_01624_b200 import synth
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    out = long_sequence_paths(pkg, synth, dev, torch.cuda.current_stream(), args.warmup, max(args.steps, 10))
    out["peaks"] = measured_peaks()
    print(json.dumps(out))


def run_macro_step(args, pkg, synth, wl, step, sharded, dist, world, rank, dev, data0, lin_idx, rest_idx, bufs, stream):
    """One macro-step: M microbatches (per rank) clipped and summed into the fp32 accumulators, then noise and the
    AdamW update once.  The microbatches rotate over a small pool of distinct resident inputs (drawing 32 GB per
    microbatch is not part of the path).  Device-timed from the first norm kernel to the end of the update."""
    ws, ws_rest, sq, clip = bufs
    M = args.macro_microbatches
    pool = [data0] + [synth.generate(wl, seed=1000 + rank, device=dev, microbatch=k)
                      for k in range(1, max(1, min(args.pool, M)))]
    lists = []
    for d in pool:
        ll = step.layer_list(d)
        lists.append((pkg.LayerList([ll.layers[k] for k in lin_idx]), pkg.LayerList([ll.layers[k] for k in rest_idx])))

    def microbatch(k):
        ll_lin, ll_rest = lists[k % len(lists)]
        pkg.dp_per_example_sqnorms(ll_lin, sq, False, ws)
        pkg.dp_per_example_sqnorms(ll_rest, sq, True, ws_rest)
        pkg.dp_clip_factors(sq, wl.C, clip)
        pkg.dp_clipped_accumulate(ll_lin, clip, ws)
        pkg.dp_clipped_accumulate_after_sqnorms(ll_rest, clip, ws_rest)

    def finish():
        step.examples_seen = wl.B * M * world
        if sharded is None:
            step.finish_macro_batch()
        else:
            sharded.finish_macro_batch()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for k in range(max(args.warmup, 3)):
        microbatch(k)
    finish()
    barrier()
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    l0 = pkg.dp_launch_count()
    t0, t1, t1b, t2 = (torch.cuda.Event(enable_timing=True) for _ in range(4))
    barrier()
    t0.record(stream)
    for k in range(M):
        microbatch(k)
    t1.record(stream)
    launches = pkg.dp_launch_count() - l0
    verify = None
    if args.verify:
        # Untimed: the accumulator after M microbatches against count_p x (one pass over pool entry p), summed in
        # fp64; and the bound ||sum of clipped gradients|| <= N C that clipping guarantees.
        acc_loop = step.acc.clone()
        ref = torch.zeros(step.n_flat, dtype=torch.float64, device=dev)
        for p_ in range(len(lists)):
            step.acc.zero_()
            microbatch(p_)
            ref += step.acc.double() * float(len(range(p_, M, len(lists))))
        step.acc.copy_(acc_loop)
        diff = float((acc_loop.double() - ref).norm() / ref.norm())
        norm = float(acc_loop.double().norm())
        verify = {"rel_l2_vs_counted_single_passes": diff, "acc_norm": norm, "bound_N_times_C": wl.B * M * wl.C,
                  "within_bound": bool(norm <= wl.B * M * wl.C * (1 + 1e-3))}
        del acc_loop, ref
    l1 = pkg.dp_launch_count()
    t1b.record(stream)
    finish()
    t2.record(stream)
    barrier()
    launches += pkg.dp_launch_count() - l1
    clocks = sampler.stop()
    if pkg.dp_poll_status() != 0:
        raise RuntimeError("device status not clean after the macro-step")
    upd_ms = t1b.elapsed_time(t2)
    total_ms = t0.elapsed_time(t1) + upd_ms
    if dist is not None:
        t = torch.tensor([total_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    if rank == 0:
        N = wl.B * M * world
        name = "bert_large_megabatch" if M == 8192 and args.blocks == 24 else \
            f"bert_large x {M} microbatches" + ("" if args.blocks == 24 else f" [first {args.blocks} blocks only]")
        print(json.dumps({
            "metric": METRIC, "value": N / (total_ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": 1,
            "warmup": max(args.warmup, 3), "ms_per_step": total_ms, "macro_step_s": total_ms * 1e-3,
            "update_ms": upd_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": name, "B": wl.B, "T": wl.T, "microbatches_per_step": M, "examples_per_step": N,
                       "resident_microbatch_pool": len(lists), "params": wl.n_params(), "parallelism": f"dp{world}",
                       "l2": "inputs (32 GB per microbatch) far exceed L2; no flush"},
            "verify": verify, "gpu_launches": int(launches), "clocks": clocks}))


def run_e2e(pkg, synth, wl, data, one_step, make_lists, clip, stream, n_steps):
    """Same step through the public API with HOST buffers: every step copies all of its layer inputs from pinned
    host memory to the device and reads the clip factors back.  The inputs of step k + 1 are copied (on a second
    stream, into a second set of device buffers) while step k computes, as a training loop would prefetch them;
    the link is the bound either way (32 GB per step)."""
    host = []
    try:
        for ld in data:
            host.append([None if t is None else torch.empty(t.shape, dtype=t.dtype, pin_memory=True).copy_(t)
                         for t in (ld.A, ld.G, ld.ids)])
        mirror = "full pinned mirror of every layer's inputs; two device input sets, copy of step k+1 under step k"
        sets = [data, [synth.LayerData(ld.spec, G=torch.empty_like(ld.G), A=None if ld.A is None else torch.empty_like(ld.A),
                                       ids=None if ld.ids is None else torch.empty_like(ld.ids)) for ld in data]]
    except RuntimeError:
        return None
    lists = [None, make_lists(sets[1])]
    clip_h = torch.empty(clip.shape, dtype=clip.dtype, pin_memory=True)
    h2d = sum(t.numel() * t.element_size() for h in host for t in h if t is not None)
    d2h = clip_h.numel() * clip_h.element_size()
    copier = torch.cuda.Stream()
    copied = [torch.cuda.Event(), torch.cuda.Event()]
    done = [torch.cuda.Event(), torch.cuda.Event()]

    def copy_in(k):          # inputs of step k into set k % 2, once the step that last used that set has finished
        with torch.cuda.stream(copier):
            copier.wait_event(done[k % 2])
            for ld, h in zip(sets[k % 2], host):
                for dst, src in zip((ld.A, ld.G, ld.ids), h):
                    if dst is not None:
                        dst.copy_(src, non_blocking=True)
            copied[k % 2].record(copier)

    def compute(k):
        stream.wait_event(copied[k % 2])
        one_step(lists=lists[k % 2])
        clip_h.copy_(clip, non_blocking=True)
        done[k % 2].record(stream)

    def run(n):
        for ev in done:
            ev.record(stream)
        copy_in(0)
        for k in range(n):
            if k + 1 < n:
                copy_in(k + 1)
            compute(k)
            stream.synchronize()      # the host reads the step's result before it goes on

    run(1)
    torch.cuda.synchronize()
    a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    run(n_steps)
    b_.record(stream)
    torch.cuda.synchronize()
    ms = a.elapsed_time(b_) / n_steps
    return {"value": wl.B / (ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
            "ms_per_step": ms, "steps": n_steps, "host_buffers": mirror}


if __name__ == "__main__":
    main()
