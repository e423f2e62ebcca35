#!/usr/bin/env python
"""Benchmark of the batched verification step (one step = one sled_verify_batch over a batch of
synthetic device requests, commit / rollback included).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
                    [--shape llama8b] [--batch 16] [--layers L] [--greedy]

Prints ONE JSON line.  Metric: verified (committed) tokens per second at the Llama-3-8B shape.
`value` is measured with the draft distributions already in device memory, `e2e` with them in
pinned host memory (copied in and results copied out inside the timed region).  `roofline` is for
the tensor-core linear-layer kernel, the dominant one.  `--impl reference` times the CPU oracle.
Under torchrun every rank runs its own replica on its own requests (no data-path collective).
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
from dataclasses import replace

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2506_09397_b200 import inputs as I

# DRAM traffic of the linear-layer kernel per launch (ncu: dram__bytes_read.sum + dram__bytes_write.sum, summed over
# the 129 launches of a step; profiles/ncu_linear_and_attention_kernels_llama8b_2layer_b{16,64}.txt), keyed by
# (shape, layers, batch).  Only valid for the kernel source it was taken from: reported as null when that file has
# changed since.
TRAFFIC_LINEAR = {"bytes_per_launch": {("llama8b", 32, 16): 119.4e6, ("llama8b", 32, 64): 127.7e6},
                  "source_sha1": "34e4a651329b36d0406bc42b191d7a0961ff9274"}

METRIC = "verified_tokens_per_s"
UNIT = "tokens/s"


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="sled", choices=["sled", "reference"])
    ap.add_argument("--shape", default="llama8b", choices=sorted(I.SHAPES))
    ap.add_argument("--batch", type=int, default=16)
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (small captures for ncu)")
    ap.add_argument("--greedy", action="store_true")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--workload", default="step", choices=["step", "accept", "attention"],
                    help="step: the full verification step (the headline); accept / attention: one kernel alone "
                         "on the acceptance-only / attention-only workload")
    ap.add_argument("--tau", type=float, default=1.0)
    return ap.parse_args(argv)


def workload(args, rank: int):
    """Per-rank batch description: draft lengths and context lengths (seeded by rank)."""
    shape = I.SHAPES[args.shape]
    if args.layers:
        shape = replace(shape, n_layers=args.layers)
    seed = args.seed + 1000 * rank
    if shape.name == "llama1b":
        ks = I.draw_k(args.batch, [2, 3, 4, 5, 6, 7, 8], seed)
        ctx = I.draw_context_lengths(args.batch, 256, 2048, seed)
    elif shape.name == "llama8b":
        ks = I.draw_k(args.batch, [3, 5, 8], seed)
        ctx = I.draw_context_lengths(args.batch, 512, 4096, seed)
    else:
        ks = I.draw_k(args.batch, [2, 4, 8], seed)
        ctx = I.draw_context_lengths(args.batch, 32, 256, seed)
    return shape, ks, ctx, seed


def workload_name(args, shape, ks, ctx):
    return (f"{shape.name} ({shape.n_layers} layers) full verify step, B={args.batch}, k_i in {sorted(set(ks))}, "
            f"contexts {min(ctx)}..{max(ctx)}, {'greedy' if args.greedy else 'sampling tau=1.0'}")


# ------------------------------------------------------------------ clocks --
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows = []
        self.proc = None
        self.gpu = gpu_index

    def start(self):
        # NVML from a thread (a sample every 10 ms from the first millisecond on); nvidia-smi as the fallback, whose
        # start-up alone can outlast a short timed region
        self.stop_flag = False
        try:
            import pynvml
            pynvml.nvmlInit()
            try:
                uuid = str(torch.cuda.get_device_properties(self.gpu).uuid)
                h = pynvml.nvmlDeviceGetHandleByUUID(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
            except Exception:
                h = pynvml.nvmlDeviceGetHandleByIndex(self.gpu)
            mx = pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM)
            bits = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4}

            def poll():
                while not self.stop_flag:
                    try:
                        clk = pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)
                        try:
                            r = pynvml.nvmlDeviceGetCurrentClocksEventReasons(h)
                        except Exception:
                            r = pynvml.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                        self.rows.append([str(self.gpu), str(clk), str(mx), "", ""] +
                                         ["Active" if r & bits[n] else "Not Active" for n in
                                          ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")])
                    except Exception:
                        pass
                    time.sleep(0.01)

            self.thread = threading.Thread(target=poll, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.thread = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(self.gpu)], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        self.stop_flag = True
        if getattr(self, "thread", None):
            self.thread.join(timeout=1)
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
        sm, mx, reasons = [], 0.0, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[1]))
                mx = max(mx, float(r[2]))
                for name, val in zip(names, r[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            except Exception:
                pass
        busy = [x for x in sm if x > 0]
        return {"sm_mhz": statistics.median(busy) if busy else None, "sm_max_mhz": mx or None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------ algorithmic work --
def linear_shapes(shape):
    s = shape
    qd, kd = s.n_q_heads * s.head_dim, s.n_kv_heads * s.head_dim
    per_layer = [(qd + 2 * kd, s.d_model), (s.d_model, qd), (2 * s.ffn_dim, s.d_model), (s.d_model, s.ffn_dim)]
    return per_layer * s.n_layers + [(s.vocab, s.d_model)]


def linear_bytes(shape, T: int) -> float:
    """Bytes the linear layers must move in one step: every weight once (bf16), their bf16 inputs,
    their fp32 outputs."""
    es = 2 if shape.weight_dtype == "bf16" else 4
    return float(sum(n * k * es + T * k * es + T * n * 4 for n, k in linear_shapes(shape)))


def linear_flops(shape, T: int) -> float:
    return 2.0 * T * shape.streamed_params()


def step_bytes(shape, ks, ctx, n_reject: int) -> float:
    """All bytes one step must move: weights, KV read and written, logits written and read,
    one draft-distribution row per rejecting request."""
    T = sum(k + 1 for k in ks)
    kvb = shape.kv_bytes_per_token()
    return (linear_bytes(shape, T) + sum(c + k + 1 for c, k in zip(ctx, ks)) * kvb + T * kvb
            + T * shape.vocab * 4 + n_reject * shape.vocab * 4)


# ------------------------------------------------------------------ oracle arm --
def oracle_sample_time(shape, weights_host, ks, ctx, seed, which: int, greedy: bool):
    """Times the CPU oracle on request `which` of the batch.  Returns (seconds, committed tokens, threads)."""
    from oracle import oracle as O
    conv = lambda t: t.numpy() if t.dtype == torch.float32 else t
    w = {k: [conv(t) for t in v] if isinstance(v, list) else conv(v) for k, v in weights_host.items()}
    orc = O.OracleModel(shape, w)
    K, V = I.make_kv(shape, ctx[which], seed, which)
    orc.load_kv(which, K.float().numpy(), V.float().numpy(), pending=1)
    del K, V
    d, q = I.make_drafts(shape.vocab, ks[which], seed, which)
    t0 = time.perf_counter()
    st, n_acc, nxt, _, _ = orc.verify(which, d.numpy(), None if greedy else q.numpy(), seed, 1.0, greedy)
    return time.perf_counter() - t0, n_acc + 1, O.num_threads()


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    shape, ks, ctx, seed = workload(args, 0)
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    w = I.weights_to(I.make_weights(shape, seed, device=dev), "cpu")
    which = int(np.argmin(ks))
    times, toks, threads = [], 0, 1
    for i in range(args.warmup + args.steps):
        dt, n_tok, threads = oracle_sample_time(shape, w, ks, ctx, seed, which, args.greedy)
        if i >= args.warmup:
            times.append(dt)
            toks += n_tok
    total = sum(times)
    value = toks / total
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "impl": "reference",
            "config": {"workload": workload_name(args, shape, ks, ctx)},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                             "sample": f"each step = request {which} of the batch alone (k={ks[which]}, "
                                       f"context {ctx[which]}), 1 of {args.batch} requests"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# -------------------------------------------------------------------- sled arm --
def aggregate(local_tokens: float, local_ms: float, world: int):
    """Whole-job numbers from per-rank ones: tokens add up, the time is the slowest rank's."""
    if world == 1:
        return local_tokens, local_ms
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([local_tokens], dtype=torch.float64, device=dev)
    m = torch.tensor([local_ms], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    dist.all_reduce(m, op=dist.ReduceOp.MAX)
    return float(t.item()), float(m.item())


def run_sled(args):
    from paper_2506_09397_b200 import binding as B
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the verification path has no CPU implementation")
    torch.cuda.set_device(local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    shape, ks, ctx, seed = workload(args, rank)
    Bn = args.batch
    T = sum(k + 1 for k in ks)
    dev = f"cuda:{local_rank}"

    w = I.make_weights(shape, seed, device=dev)
    n_pages = sum((c + k + 1 + 15) // 16 for c, k in zip(ctx, ks)) + 64
    stream = torch.cuda.Stream(device=dev)
    eng = B.Engine(shape, w, n_pages=n_pages, max_batch=Bn, max_k=max(ks), max_step_tokens=max(T, 16),
                   temperature=1.0, greedy=args.greedy, device_index=local_rank, stream=stream.cuda_stream)
    need_host_w = (rank == 0 and world == 1 and not args.no_cpu_baseline)
    w_host = I.weights_to(w, "cpu") if need_host_w else None
    del w
    torch.cuda.empty_cache()
    eng.shuffle_pages(seed)
    for i in range(Bn):
        K, V = I.make_kv(shape, ctx[i], seed, i, device=dev)
        eng.load_kv(i, K, V, pending=1)
        del K, V
    drafts_host, q_dev, q_host = [], [], []
    for i in range(Bn):
        d, q = I.make_drafts(shape.vocab, ks[i], seed, i, device=dev)
        drafts_host.append(np.ascontiguousarray(d.cpu().numpy()))
        q_dev.append(q)
        if not args.no_e2e:
            q_host.append(q.cpu().pin_memory())
    torch.cuda.synchronize()

    def marshal(qs):
        reqs = (B.SledRequest * Bn)()
        for i in range(Bn):
            reqs[i].ctx_id = i
            reqs[i].draft_tokens = drafts_host[i].ctypes.data
            reqs[i].draft_probs = None if args.greedy else qs[i].data_ptr()
            reqs[i].k = ks[i]
        return reqs

    res = (B.SledResult * Bn)()
    L = B.lib()

    def one_step(reqs, step_seed):
        rc = eng.verify_batch_raw(reqs, Bn, step_seed, res)
        if rc != 0:
            raise SystemExit(f"sled_verify_batch failed: {B.strerror(rc)}")
        committed = 0
        for i in range(Bn):
            if res[i].status != 0:
                raise SystemExit(f"request {i} came back with status {res[i].status}")
            committed += res[i].n_accepted + 1
            L.sled_debug_truncate(eng.h, i, ctx[i], 1)   # same state for every step (host bookkeeping only)
        return committed

    def timed(reqs, steps, warmup):
        for s in range(warmup):
            one_step(reqs, 100 + s)
        launches0 = eng.stats().kernels_launched
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        committed = 0
        e0.record(stream)
        for s in range(steps):
            committed += one_step(reqs, 1000 + s)
        e1.record(stream)
        torch.cuda.synchronize()
        if world > 1:
            torch.distributed.barrier()
        return committed, e0.elapsed_time(e1), eng.stats().kernels_launched - launches0

    sampler = ClockSampler(local_rank)
    sampler.start()
    reqs_dev = marshal(q_dev)
    committed, ms, launches = timed(reqs_dev, args.steps, args.warmup)
    tok_all, ms_all = aggregate(float(committed), ms, world)
    value = tok_all / (ms_all / 1e3)

    e2e = None
    if not args.no_e2e:
        reqs_host = marshal(q_host)
        c2, ms2, _ = timed(reqs_host, args.steps, args.warmup)
        t2, m2 = aggregate(float(c2), ms2, world)
        h2d = 0 if args.greedy else sum(k * shape.vocab * 4 for k in ks)
        e2e = {"value": t2 / (m2 / 1e3), "unit": UNIT, "h2d_bytes_per_step": h2d + 64 * T,
               "d2h_bytes_per_step": 12 * Bn, "ms_per_step": m2 / args.steps}

    clocks = sampler.stop()   # sampled over the warm-up and timed steps of both measurements

    # device time per kernel kind (events between kernels; extra steps, not the ones behind `value`)
    eng.set_timing(True)
    lin_ms, attn_ms, acc_ms, oth_ms, step_ms = [], [], [], [], []
    n_rej = 0
    for s in range(5):
        one_step(reqs_dev, 2000 + s)
        st = eng.stats()
        lin_ms.append(st.ms_linear); attn_ms.append(st.ms_attention); acc_ms.append(st.ms_accept)
        oth_ms.append(st.ms_other); step_ms.append(st.ms_step)
        n_rej = sum(1 for i in range(Bn) if res[i].n_accepted < ks[i])
    eng.set_timing(False)
    st = eng.stats()
    n_lin = st.linear_launches_last_step
    lin = statistics.median(lin_ms)
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    hbm_peak = peaks.get("hbm_gbs", 6650.0)
    tc_peak = peaks.get("bf16_tflops_sustained", 1400.0)
    peak_src = "measured" if peaks else "fallback"
    lb, lf = linear_bytes(shape, T), linear_flops(shape, T)
    if lb / (hbm_peak * 1e9) >= lf / (tc_peak * 1e12):
        ach = lb / (lin / 1e3) / 1e9
        roof = {"bound": "hbm", "achieved": ach, "peak": hbm_peak, "unit": "GB/s", "frac": ach / hbm_peak}
    else:
        ach = lf / (lin / 1e3) / 1e12
        roof = {"bound": "tensor", "achieved": ach, "peak": tc_peak, "unit": "TFLOP/s", "frac": ach / tc_peak}
    traffic = None
    try:
        import hashlib
        src = open(os.path.join(ROOT, "paper_2506_09397_b200", "csrc", "gemm_tc.cu"), "rb").read()
        if hashlib.sha1(src).hexdigest() == TRAFFIC_LINEAR["source_sha1"]:
            traffic = TRAFFIC_LINEAR["bytes_per_launch"].get((shape.name, shape.n_layers, Bn))
    except Exception:
        pass
    roof.update({"traffic": traffic, "algorithmic_bytes_per_launch": lb / max(n_lin, 1), "kernel": "linear-layer kernel (all linear layers of a step)", "peak_source": peak_src,
                 "launches_per_step": n_lin, "avg_launch_ms": lin / max(n_lin, 1),
                 "algorithmic_bytes_per_step": lb, "algorithmic_flops_per_step": lf})
    sb = step_bytes(shape, ks, ctx, n_rej)
    step_s = ms_all / args.steps / 1e3
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_all / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if shape.weight_dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": workload_name(args, shape, ks, ctx), "tokens_scored_per_step": T,
                       "l2": "inputs larger than L2 (a step streams %.2f GB of weights)" % (2e-9 * shape.streamed_params()),
                       "draft_distributions": "independent of the target (softmax of N(0,1) logits)",
                       "kv": "synthetic N(0,1) cache content in permuted 16-token pages"},
            "clocks": clocks, "gpu_launches": int(launches),
            "scored_positions_per_s": T * world / step_s,
            "acceptance_rate": (committed / args.steps - Bn) / max(sum(ks), 1),
            "step_hbm": {"algorithmic_bytes": sb, "achieved_GBps": sb / step_s / 1e9,
                         "frac_of_hbm_peak": sb / step_s / 1e9 / hbm_peak, "peak_source": peak_src},
            "kernel_ms": {"linear": lin, "attention": statistics.median(attn_ms), "accept": statistics.median(acc_ms),
                          "other": statistics.median(oth_ms), "step_with_events": statistics.median(step_ms)},
            "roofline": roof}
    if e2e:
        line["e2e"] = e2e
    if need_host_w:
        which = int(np.argmin(ks))
        dt, n_tok, threads = oracle_sample_time(shape, w_host, ks, ctx, seed, which, args.greedy)
        line["cpu_baseline"] = {"value": n_tok / dt, "unit": UNIT, "cores": threads, "kind": "oracle", "seconds": dt,
                                "sample": f"request {which} of the batch alone (k={ks[which]}, context {ctx[which]}), "
                                          f"1 of {Bn} requests, one pass"}
    eng.shutdown()
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()


def _peaks():
    try:
        return json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json"))), "measured"
    except Exception:
        return {"hbm_gbs": 6650.0, "bf16_tflops_sustained": 1400.0}, "fallback"


def run_accept_only(args):
    """Acceptance kernel alone: 512 requests x (7 drafts + 1 bonus) rows over the 128256-entry vocabulary."""
    from paper_2506_09397_b200 import binding as B
    n, k, V = 512, 7, 128256
    z, q, d = I.make_accept_rows(n, k, V, tau_draft=1.0, seed=args.seed, device="cuda")
    logits, qrows = z.reshape(n * (k + 1), V), q.reshape(n * k, V)
    cu = [8 * i for i in range(n + 1)]
    ctx = [10_000 + i for i in range(n)]
    pos0 = [100 + (i % 37) for i in range(n)]
    dh = d.cpu().numpy().reshape(-1)
    times, got = [], None
    for it in range(args.warmup + args.steps):
        got, ms = B.accept_rows(logits, cu, dh, None if args.greedy else qrows, ctx, pos0, args.tau, args.greedy, seed=it)
        if it >= args.warmup:
            times.append(ms)
    ms = statistics.median(times)
    rows_read = sum(g[0] + 1 for g in got)                     # rows up to and including the deciding one
    n_rej = sum(1 for g in got if g[0] < k)
    alg = rows_read * V * 4 + (0 if args.greedy else n_rej * V * 4)
    peaks, src = _peaks()
    ach = alg / (ms / 1e3) / 1e9
    print(json.dumps({"metric": "acceptance_rows_per_s", "value": rows_read / (ms / 1e3), "unit": "rows/s", "n_gpus": 1,
                      "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
                      "dtype": "f32/u64", "data": "synthetic",
                      "config": {"workload": f"acceptance only: 512 requests x 8 rows, V=128256, tau={args.tau}, "
                                             f"{'greedy' if args.greedy else 'sampling'}; {rows_read} rows examined",
                                 "l2": "inputs larger than L2 (2.1 GB of logits)"},
                      "acceptance_rate": sum(g[0] for g in got) / (n * k),
                      "roofline": {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                   "frac": ach / peaks["hbm_gbs"], "traffic": None, "peak_source": src,
                                   "algorithmic_bytes": alg, "all_rows_bytes": n * (k + 1) * V * 4}}))


def run_attention_only(args):
    """Attention kernel alone: 256 requests, query length 2..9, lognormal cache lengths, 32/8 heads of 128."""
    from paper_2506_09397_b200 import binding as B
    shape = I.ModelShape("attn_only", 1, 64, 32, 8, 128, 64, 64, 5e5, "bf16", "bf16")
    nreq = 256
    qlens = [int(x) for x in torch.randint(2, 10, (nreq,), generator=torch.Generator().manual_seed(1))]
    lens = I.draw_lognormal_kv_lengths(nreq, 2048, 1.0, 128, 16384, args.seed + 1)
    w = I.make_weights(shape, 0)
    eng = B.Engine(shape, w, n_pages=sum((n + 15) // 16 for n in lens) + 8, max_batch=nreq, max_k=8,
                   max_step_tokens=sum(qlens))
    eng.shuffle_pages(2)
    for i, n in enumerate(lens):
        K, V = I.make_kv(shape, n, 6, i, device="cuda")
        eng.load_kv(i, K, V, pending=0)
    T = sum(qlens)
    q = torch.randn(T, 32, 128, device="cuda").to(torch.bfloat16)
    out = torch.zeros_like(q)
    times = []
    for it in range(args.warmup + args.steps):
        ms = eng.attention_ragged(0, list(range(nreq)), qlens, q, out)
        if it >= args.warmup:
            times.append(ms)
    ms = statistics.median(times)
    alg = sum(lens) * 2 * 8 * 128 * 2 + 2 * T * 32 * 128 * 2
    flops = 4.0 * 32 * 128 * sum(ql * (n - ql) + ql * (ql + 1) / 2 for n, ql in zip(lens, qlens))
    peaks, src = _peaks()
    ach = alg / (ms / 1e3) / 1e9
    print(json.dumps({"metric": "attention_cached_tokens_per_s", "value": sum(lens) / (ms / 1e3), "unit": "tokens/s",
                      "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
                      "dtype": "bf16", "data": "synthetic",
                      "config": {"workload": f"attention only: 256 requests, q_len 2..9, cache lengths lognormal "
                                             f"(median 2048, sigma 1, 128..16384; mean {sum(lens) / nreq:.0f}), "
                                             "32/8 heads of 128, permuted 16-token pages",
                                 "l2": "inputs larger than L2 (%.2f GB of cache)" % (alg / 1e9)},
                      "tflops": flops / (ms / 1e3) / 1e12,
                      "roofline": {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                   "frac": ach / peaks["hbm_gbs"], "traffic": None, "peak_source": src,
                                   "algorithmic_bytes": alg}}))
    eng.shutdown()


def main(argv=None):
    args = parse_args(argv)
    if args.impl == "reference":
        run_reference(args)
    elif args.workload == "accept":
        run_accept_only(args)
    elif args.workload == "attention":
        run_attention_only(args)
    else:
        run_sled(args)


if __name__ == "__main__":
    main()
