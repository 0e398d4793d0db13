#!/usr/bin/env python
"""Benchmark of the parallelised ZO estimator step (one zo_step = one pass of the whole hot path:
shared prefix, 2q-replica MP-LoRA forward, 2q losses, q projected gradients, ZO-SGD update).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload llama7b] [--impl ours|reference]

Prints one JSON line.  `value` = perturbed-forward tokens/s = 2q*E*S*steps / device time, inputs
resident in HBM; `e2e` = the same through zo_step_host (tokens/labels copied from pinned host memory,
losses read back every step).  N > 1 runs N independent replicas of the job (the path is not sharded).
"""
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

from workloads import config, make_decoder_globals, make_decoder_layer, make_linear_problem  # noqa: E402
from workloads.spec import ARCH_LINEAR, ARCH_OPT  # noqa: E402

METRIC, UNIT = "perturbed_fwd_tokens_per_s", "tokens/s"

# DRAM bytes (read + write) per token row of one gate|up launch of the tensor-core GEMM, from an ncu
# capture (dram__bytes_read.sum + dram__bytes_write.sum) of that launch at 8192 token rows; activations,
# outputs and one weight-panel read per raster group all grow with the rows, so a full launch is scaled
# by rows.  None = the kernel changed since the counters were taken.
GEMM_FC1_DRAM_BYTES_PER_ROW = {"llama7b": 117485.0}   # (791.41 + 171.03) MB / 8192 rows


def hbm_kernel_rates(spec, prof, peaks, steps):
    """{class: {ms and GB per step, GB/s, frac of the measured copy peak}} for the classes the library books bytes for;
    the LoRA down-projection is booked in flops 2*rows*J*K and reads rows*K elements."""
    out = {}
    es = 2 if spec.bf16 else 4
    for k in ("attention", "norm", "lora_apply", "rope", "lora_down"):
        ms, work, cnt = prof.get(k, (0.0, 0.0, 0))
        if not cnt or ms <= 0 or work <= 0:
            continue
        if k == "lora_down":
            work = work / (2.0 * (spec.n_targets if spec.arch != 0 else 1) * spec.lora_rank) * es
        gbs = work / (ms * 1e-3) / 1e9
        out[k] = {"ms_per_step": round(ms / steps, 3), "launches_per_step": cnt // steps,
                  "GB_per_step": round(work / steps / 1e9, 3), "GB/s": round(gbs, 1),
                  "frac": round(gbs / peaks["hbm_gbs"], 3) if peaks.get("hbm_gbs") else None}
    return out


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], tflops=p["bf16_tflops"], tflops_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, tflops=1590.0, tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap,power.draw")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "200"], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=lambda: self.lines.extend(self.proc.stdout), daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        self.thread.join(timeout=2)
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for nm, v in zip(names, f[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
            try:
                pw.append(float(f[6]))
            except (IndexError, ValueError):
                pass
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons), "power_w": float(np.median(pw)) if pw else None}


def max_over_ranks(values, device):
    """Slowest rank's figure for each entry of `values` (the job is N independent replicas of the
    step, so whole-job throughput = N * units per step / the slowest rank's time)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return list(values)
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def rank_command(n, argv):
    """Command line that starts n ranks of this script on one node (one process per GPU, rendezvous on
    the loopback address), as the launcher of `--gpus n` does when no launcher started us."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *argv]


def timed_region(step, steps, barrier, stamp):
    """Exactly `steps` calls of step(i) between two barriers; the time between the two stamps in ms.
    `barrier()` lines the ranks up and drains the device; `stamp()` returns an object with
    elapsed_time(later_stamp) in ms (a CUDA event on the launching stream)."""
    barrier()
    t0 = stamp()
    for i in range(steps):
        step(i)
    t1 = stamp()
    barrier()
    return t0.elapsed_time(t1)


def whole_job_value(world, units_per_step, steps, ms):
    return world * units_per_step * steps / (ms * 1e-3)


def load_problem(spec, seed=1234, b_std=0.01, weights=None):
    """Synthetic weights on the device, one decoder block in host memory at a time; `weights` =
    "int8" / "nf4" stores the four linear weights of every block in that weight-only format."""
    import paper_2409_15520_b200 as zo
    from workloads import quantize_layer
    if spec.arch == ARCH_LINEAR:
        return zo.DeviceProblem(make_linear_problem(spec, seed=seed, b_std=b_std), spec.bf16)
    p = make_decoder_globals(spec, seed)
    mk = (lambda l: make_decoder_layer(spec, seed, l, b_std)) if not weights else \
        (lambda l: quantize_layer(make_decoder_layer(spec, seed, l, b_std), weights))
    p["layers"] = (mk(l) for l in range(spec.n_layers))
    return zo.DeviceProblem(p, spec.bf16, n_layers=spec.n_layers)


def algorithmic_flops_per_step(spec):
    """GEMM flops the method must do per step (nothing saved by sharing is counted as done):
    per replica row and layer 2*(4 d^2 + c d ffn), LM head on labelled rows, LoRA terms."""
    n, T = 2 * spec.q, spec.E * spec.S
    if spec.arch == ARCH_LINEAR:
        return 2.0 * T * spec.d_model * spec.d_out
    d, f = spec.d_model, spec.d_ffn
    c = 2 if spec.arch == ARCH_OPT else 3
    per_row = 2.0 * (4 * d * d + c * d * f)
    return per_row * spec.n_layers * n * T + 2.0 * n * spec.E * spec.n_labelled * d * spec.vocab


def oracle_sample(spec, seed=1234):
    """Bounded CPU sample of the same workload: the oracle's two perturbed forward passes of one query
    (q = 1, the +/- pair) on up to eight sequences of the batch through a 2-block copy of the model.
    The decoder blocks and the loss head (final norm, LM head, cross-entropy on the labelled rows) are
    timed apart, so only the blocks' time is scaled to the full depth.
    Returns (seconds of the sample, seconds scaled to the full model, token-forwards done, description)."""
    import oracle
    from oracle.model import decoder_hidden, row_losses
    from oracle.zo import draw_z
    if spec.arch == ARCH_LINEAR:
        small = spec.with_(q=1)
        p = make_linear_problem(small, seed=seed, b_std=0.01)
        t0 = time.perf_counter()
        oracle.zo_step(small, p, p["X"], p["target"], 1, 1, spec.eps, spec.lr)
        dt = time.perf_counter() - t0
        return dt, dt, 2 * small.E * small.S, "q=1 on the full token block"
    L = min(2, spec.n_layers)
    Es = min(8, spec.E)                      # sized for 10-30 s of CPU work at the 7B shape
    small = spec.with_(n_layers=L, E=Es, q=1)
    p = make_decoder_globals(small, seed)
    p["layers"] = [make_decoder_layer(small, seed, l, 0.01) for l in range(L)]
    z = draw_z(small, p, 1, 0)
    t_blocks = t_head = 0.0
    for k in (+1.0, -1.0):                   # theta + k eps z, one forward pass each (Algorithm 1)
        Bn = [(np.asarray(Lr["B"], np.float64) + k * spec.eps * z[l])[None] for l, Lr in enumerate(p["layers"])]
        t0 = time.perf_counter()
        h = decoder_hidden(small, p, Bn, p["tokens"])
        t1 = time.perf_counter()
        row_losses(small, p, h, p["labels"]).mean()
        t2 = time.perf_counter()
        t_blocks += t1 - t0
        t_head += t2 - t1
    return (t_blocks + t_head, t_blocks * spec.n_layers / L + t_head, 2 * Es * small.S,
            f"q=1, {Es} sequences of {small.S} tokens, {L} of {spec.n_layers} blocks "
            f"(blocks' time scaled by depth, loss head timed apart and not scaled)")


def run_sweep(args):
    """MP-LoRA linear micro-benchmark (d_in = d_out = 4096, 4096 tokens, rank x q grid): one JSON line per
    point with the shared-input form (one base GEMM amortised over the 2q replicas, then the expand
    kernel: bound by writing 2q*T*k outputs) and the replicated-input form (one GEMM over 2q*T rows with
    the low-rank term in its epilogue: bound by the tensor pipe)."""
    import torch
    import paper_2409_15520_b200 as zo
    peaks = _peaks()
    T = k = 4096
    dev = "cuda"
    g = torch.Generator(device=dev).manual_seed(1234)
    W = (0.02 * torch.randn(k, k, device=dev, generator=g)).to(torch.bfloat16)
    bias = (0.02 * torch.randn(k, device=dev, generator=g)).to(torch.bfloat16)
    ranks = [args.rank] if args.rank else [8, 16, 64]
    qs = [args.q] if args.q else [1, 2, 4, 8, 16, 32]
    ev = lambda: torch.cuda.Event(enable_timing=True)
    for r in ranks:
        A = (0.02 * torch.randn(r, k, device=dev, generator=g)).to(torch.bfloat16)
        B = 0.01 * torch.randn(r, k, device=dev, generator=g)
        for q in qs:
            n = 2 * q
            X = torch.randn(n * T, k, device=dev, generator=g).to(torch.bfloat16)
            Y = torch.empty(n, T, k, device=dev, dtype=torch.bfloat16)
            out = {"r": r, "q": q, "replicas": n}
            for mode, x_rep in (("shared_input", 0), ("replicated_input", 1)):
                call = lambda: zo.mp_lora_linear(X, W, bias, A, B, T, q, 1.0, 7, 0, 1e-3, x_rep,
                                                 flags=args.flags, out=Y, sync=False)
                for _ in range(3):
                    call()
                torch.cuda.synchronize()
                e0, e1 = ev(), ev()
                reps = max(3, min(20, 64 // n))
                e0.record()
                for _ in range(reps):
                    call()
                e1.record()
                torch.cuda.synchronize()
                ms = e0.elapsed_time(e1) / reps
                flops = 2.0 * (n if x_rep else 1) * T * k * k
                out[mode] = {"ms": round(ms, 4), "gemm_tflops": round(flops / (ms * 1e-3) / 1e12, 1),
                             "frac_of_bf16_peak": round(flops / (ms * 1e-3) / 1e12 / peaks["tflops"], 3),
                             "out_gbs": round(n * T * k * 2 / (ms * 1e-3) / 1e9, 1),
                             "frac_of_hbm_peak": round(n * T * k * 2 / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], 3),
                             "tokens_per_s": round(n * T / (ms * 1e-3))}
            out["replicated_over_shared_time"] = round(out["replicated_input"]["ms"] / out["shared_input"]["ms"], 2)
            print(json.dumps(out), flush=True)


def run_ablation(args, spec):
    """The paper's runtime ablations on this GPU (fixed-length synthetic batches on the 7B shape):
    inner-loop (q = 1: the +/- pair in one pass vs two sequential passes) over seq x batch, and
    outer-loop (q*E = 16 fixed) over (q, E) x seq, each under the schedules that apply.  One JSON
    line per point, ms per step (median of 5 after 2 warm-ups) and ratios."""
    import torch
    import paper_2409_15520_b200 as zo
    from workloads import next_token_labels
    big = spec.with_(q=16, E=16, S=256)
    prob = load_problem(big, weights=args.weights)
    est = zo.Estimator(zo.make_config(big, flags=args.flags, weight_format=args.weights))
    rng = np.random.default_rng(7)

    def time_point(q, E, S, schedule):
        tok = rng.integers(0, spec.vocab, size=(E, S), dtype=np.int32)
        lab = next_token_labels(tok, min(spec.n_labelled, S - 1))
        dt, dl = torch.tensor(tok, device="cuda"), torch.tensor(lab, device="cuda")
        est.set_schedule(schedule)
        ts = []
        for i in range(7):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            est.step(prob, E, S, 50 + i, q, spec.eps, spec.lr, tokens=dt, labels=dl)
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        est.losses()
        return float(np.median(ts[2:]))

    for S in (64, 128, 256):
        for E in (1, 8, 16):
            par, seq = time_point(1, E, S, "full"), time_point(1, E, S, "sequential")
            print(json.dumps({"table": "inner_loop", "weights": args.weights or "bf16", "q": 1, "seq": S, "batch": E, "ms_parallel_pair": round(par, 3),
                              "ms_sequential_pair": round(seq, 3), "speedup": round(seq / par, 3)}), flush=True)
    if args.weights:
        return                      # the paper's quantisation figure is the inner-loop grid only
    for S in (64, 128, 256):
        for q, E in ((1, 16), (4, 4), (16, 1)):
            r = {"table": "outer_loop", "q": q, "E": E, "seq": S}
            for sched in ("full", "outer_only", "inner_only", "sequential"):
                r["ms_" + sched] = round(time_point(q, E, S, sched), 3)
            r["speedup_full_vs_sequential"] = round(r["ms_sequential"] / r["ms_full"], 3)
            print(json.dumps(r), flush=True)


def run_varlen(args, spec):
    """Padding study (the paper's second argument for small E): the same E variable-length sequences
    (lengths uniform in [S/4, S]) run (a) padded to S in the fixed-length step and (b) packed back to
    back through zo_step_varlen, which spends nothing on padding rows.  One JSON line."""
    import torch
    import paper_2409_15520_b200 as zo
    from workloads import make_ragged_batch
    prob = load_problem(spec, weights=args.weights)
    est = zo.Estimator(zo.make_config(spec, flags=args.flags, weight_format=args.weights))
    toks, labs = make_ragged_batch(spec, seed=77)
    E, S, q = spec.E, spec.S, spec.q
    pad_t = np.zeros((E, S), np.int32)
    pad_l = np.full((E, S), -1, np.int32)
    for b, (t, l) in enumerate(zip(toks, labs)):
        pad_t[b, :len(t)], pad_l[b, :len(l)] = t, l
    dev = lambda a: torch.tensor(np.ascontiguousarray(a), dtype=torch.int32, device="cuda")
    d_pt, d_pl = dev(pad_t), dev(pad_l)
    d_t, d_l = dev(np.concatenate(toks)), dev(np.concatenate(labs))
    d_cu = dev(np.concatenate([[0], np.cumsum([len(t) for t in toks])]))
    real = int(sum(len(t) for t in toks))

    def timed(fn):
        ts = []
        for i in range(args.warmup + args.steps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn(i)
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        return float(np.median(ts[args.warmup:])), est.losses()[0]

    ms_pad, l_pad = timed(lambda i: est.step(prob, E, S, 7, q, spec.eps, 0.0, tokens=d_pt, labels=d_pl))
    ms_pack, l_pack = timed(lambda i: est.step_varlen(prob, d_t, d_l, d_cu, S, 7, q, spec.eps, 0.0))
    print(json.dumps({"study": "padding", "workload": args.workload, "E": E, "S": S, "q": q, "real_tokens": real,
                      "padded_tokens": E * S, "padding_fraction": round(1 - real / (E * S), 4),
                      "ms_padded": round(ms_pad, 3), "ms_packed": round(ms_pack, 3),
                      "speedup": round(ms_pad / ms_pack, 3),
                      "real_tokens_per_s_packed": round(2 * q * real / (ms_pack * 1e-3)),
                      "max_rel_loss_diff": float(np.max(np.abs(l_pad - l_pack) / np.abs(l_pad)))}))


def run_reference(args, spec):
    """The CPU oracle as it stands, timed on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import torch
    cores = torch.get_num_threads()
    for _ in range(args.warmup if args.warmup < 2 else 1):
        oracle_sample(spec)
    times = []
    for _ in range(args.steps):
        _, full, toks, what = oracle_sample(spec)
        times.append(full)
    sec = float(np.sum(times))
    value = toks * args.steps / sec
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sec / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "sample": what},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": what},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="llama7b")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--layers", type=int, default=0, help="override the depth (profiling captures of a small case)")
    ap.add_argument("--q", type=int, default=0, help="override q (profiling captures of a small case)")
    ap.add_argument("--flags", type=int, default=0, help="zo_config.flags (diagnostic kernel switches)")
    ap.add_argument("--targets", type=int, default=-1, help="override lora_targets (0 = no adapted projection)")
    ap.add_argument("--rank", type=int, default=0, help="override the LoRA rank")
    ap.add_argument("--sweep", action="store_true", help="MP-LoRA linear micro-benchmark grid (rank x q)")
    ap.add_argument("--ablation", action="store_true", help="the paper's inner/outer-loop runtime grids on this GPU")
    ap.add_argument("--varlen", action="store_true", help="padded vs packed variable-length batch (padding study)")
    ap.add_argument("--schedule", default="full", choices=["full", "outer_only", "inner_only", "sequential"],
                    help="how the step is cut into forward passes (the paper's ablation)")
    ap.add_argument("--weights", default=None, choices=["int8", "nf4"],
                    help="weight-only quantised storage of the frozen linear weights (decoded once per pass)")
    ap.add_argument("--shard-queries", action="store_true",
                    help="N > 1: spread the q queries of ONE step over the ranks (all-reduce of the 2q losses, "
                         "identical update everywhere; strong scaling) instead of N independent replicas")
    ap.add_argument("--E", type=int, default=0, help="override the number of sequences")
    ap.add_argument("--S", type=int, default=0, help="override the sequence length")
    args = ap.parse_args()
    if args.sweep:
        return run_sweep(args)
    spec = config(args.workload)
    if args.layers:
        spec = spec.with_(n_layers=args.layers)
    if args.q:
        spec = spec.with_(q=args.q)
    if args.E:
        spec = spec.with_(E=args.E)
    if args.S:
        spec = spec.with_(S=args.S, n_labelled=min(spec.n_labelled, args.S - 1))
    if args.targets >= 0:
        spec = spec.with_(lora_targets=args.targets)
    if args.rank:
        spec = spec.with_(lora_rank=args.rank)
    if args.impl == "reference":
        return run_reference(args, spec)
    if args.ablation:
        return run_ablation(args, spec)
    if args.varlen:
        return run_varlen(args, spec)

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # asked for N GPUs without a launcher around us: start the N ranks ourselves
        raise SystemExit(subprocess.call(rank_command(args.gpus, sys.argv[1:])))

    import torch
    import torch.distributed as dist
    import paper_2409_15520_b200 as zo

    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    E, S, q, eps, lr = spec.E, spec.S, spec.q, spec.eps, spec.lr
    tokens_per_step = 2 * q * E * S
    sharded = args.shard_queries
    jobs = 1 if sharded else world            # independent steps in flight across the ranks
    if sharded and world > q:
        raise SystemExit("--shard-queries needs at least one query per rank")
    # a rank that only ever runs its block of queries needs activations for that block alone
    max_shard_q = zo.query_shard(q, world, 0)[1] if sharded else 0
    prob = load_problem(spec, weights=args.weights)
    est = zo.Estimator(zo.make_config(spec, flags=args.flags, weight_format=args.weights, max_shard_q=max_shard_q))
    est.set_schedule(args.schedule)

    def one_step(seed, host=False):
        if not sharded:
            return (est.step_host if host else est.step)(prob, E, S, seed, q, eps, lr)
        begin, count = zo.query_shard(q, world, rank)
        est.set_query_shard(begin, count)
        (est.step_host if host else est.step)(prob, E, S, seed, q, eps, 0.0)
        est.set_query_shard(0, 0)
        zo.exchange_step(est.loss_buffer())
        est.apply_update(prob, seed, q, eps, lr)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def stamp():
        e = torch.cuda.Event(enable_timing=True)
        e.record()
        return e

    for i in range(max(args.warmup, 3)):
        one_step(100 + i)
    est.losses()
    # (1) the headline: K steps, no per-launch instrumentation
    sampler = ClockSampler(local)
    sampler.start()
    ms = timed_region(lambda i: one_step(1000 + i), args.steps, barrier, stamp)
    clocks = sampler.stop()
    losses, g = est.losses()
    launches = est.launch_count() * args.steps

    # (2) end to end: host tokens/labels in, losses out, every step
    def e2e_step(i):
        one_step(2000 + i, host=True)
        est.losses()
    t0 = time.perf_counter()
    ms_e2e = timed_region(e2e_step, args.steps, barrier, stamp)
    ms_e2e = max(ms_e2e, 1e3 * (time.perf_counter() - t0))
    h2d = prob.host_tokens.numel() * prob.host_tokens.element_size() + \
        prob.host_labels.numel() * prob.host_labels.element_size()
    d2h = (2 * q + q) * 4 + 4

    # (3) a second, instrumented pass (every launch bracketed by CUDA events on the launching stream) for
    # the per-kernel figures and the roofline; its events cost time, so it does not feed `value`
    prof_steps = min(args.steps, 5)
    est.profile_enable(True)
    est.profile_read()
    ms_prof = timed_region(lambda i: one_step(3000 + i), prof_steps, barrier, stamp)
    prof = est.profile_read()
    est.profile_enable(False)

    ms, ms_e2e = max_over_ranks([ms, ms_e2e], "cuda")
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = _peaks()
    gemm_classes = [k for k in prof if k.startswith("gemm_") and k != "gemm_simt"]
    gms, gfl, gcnt = (sum(prof[k][i] for k in gemm_classes) for i in range(3))
    gemm_tflops = gfl / (gms * 1e-3) / 1e12 if gms > 0 else 0.0
    inside_long_step = ms / args.steps > 200.0
    peak = peaks["tflops_sustained"] if inside_long_step else peaks["tflops"]
    total_prof = sum(v[0] for v in prof.values())
    fc1_bytes_per_row = GEMM_FC1_DRAM_BYTES_PER_ROW.get(args.workload)
    line = {
        "metric": METRIC, "value": whole_job_value(jobs, tokens_per_step, args.steps, ms), "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps,
        "higher_is_better": True, "scaling": "strong" if sharded else "weak", "vs_baseline": None,
        "dtype": "bf16" if spec.bf16 else "f32", "data": "synthetic",
        "config": {"workload": args.workload, "arch": {0: "linear", 1: "opt", 2: "llama"}[spec.arch],
                   "n_layers": spec.n_layers, "d_model": spec.d_model, "d_ffn": spec.d_ffn, "vocab": spec.vocab,
                   "lora_rank": spec.lora_rank, "q": q, "E": E, "S": S, "replicas": 2 * q,
                   "token_rows_per_step": tokens_per_step, "eps": eps, "lr": lr,
                   "l2": "inputs larger than L2 (weights and activations of several GB stream every step)",
                   "schedule": args.schedule, "weights": args.weights or "bf16",
                   "parallelism": (f"queries of one step sharded over {world} gpu(s), all-reduce of the loss array" if sharded
                                   else "replicas only" if world > 1 else "1 gpu")},
        "zo_steps_per_s": jobs * args.steps / (ms * 1e-3),
        "step_tflops": algorithmic_flops_per_step(spec) * args.steps / (ms * 1e-3) / 1e12,
        "clocks": clocks,
        # step time x median SM clock (ms x GHz = millions of SM clocks per step): separates what a change did to
        # the work per clock from what the power cap did to the clock
        "mclk_per_step": (round(ms / args.steps * clocks["sm_mhz"] / 1e3, 1)
                          if clocks.get("sm_mhz") else None),
        "e2e": {"value": whole_job_value(jobs, tokens_per_step, args.steps, ms_e2e), "unit": UNIT,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": launches,
        "roofline": {"bound": "tensor", "kernel": "gemm_tc_kernel", "achieved": gemm_tflops, "peak": peak,
                     "unit": "TFLOP/s", "frac": gemm_tflops / peak if peak else None,
                     "peak_source": f"{peaks['source']} ({'sustained' if inside_long_step else 'burst'} bf16)",
                     "frac_of_burst_peak": gemm_tflops / peaks["tflops"],
                     "frac_of_sustained_peak": gemm_tflops / peaks["tflops_sustained"],
                     "frac_of_nominal_2250": gemm_tflops / 2250.0,
                     "measured_in": f"instrumented pass of {prof_steps} steps, {ms_prof / prof_steps:.3f} ms/step",
                     "launches": gcnt, "avg_launch_ms": gms / gcnt if gcnt else None,
                     "traffic": (fc1_bytes_per_row * tokens_per_step
                                 if fc1_bytes_per_row
                                 and not (args.flags or args.rank or args.targets >= 0 or args.weights) else None),
                     "traffic_note": "gate|up launch (the largest GEMM class of the step): ncu capture of that launch at 8192 token rows, scaled by rows"},
        "gemm_tflops_by_class": {k: round(prof[k][1] / (prof[k][0] * 1e-3) / 1e12, 1)
                                 for k in gemm_classes if prof[k][0] > 0},
        # memory-bound kernels: algorithmic bytes (inputs read once, outputs written once) over their
        # CUDA-event time in the instrumented pass, against the measured copy bandwidth
        "hbm_kernels": hbm_kernel_rates(spec, prof, peaks, prof_steps),
        "kernel_time_share": {k: round(v[0] / total_prof, 4) for k, v in prof.items() if v[2]},
        "kernel_ms_per_step": {k: round(v[0] / prof_steps, 3) for k, v in prof.items() if v[2]},
        "loss_mean": float(np.mean(losses)),
    }
    if not args.no_cpu_baseline and world == 1:
        import torch as _t
        dt, full, toks, what = oracle_sample(spec)
        line["cpu_baseline"] = {"value": toks / full, "unit": UNIT, "cores": _t.get_num_threads(),
                                "kind": "oracle", "sample": what, "seconds": dt}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
