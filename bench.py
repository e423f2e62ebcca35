#!/usr/bin/env python
"""Benchmark of the batched verification step (one step = one sled_verify_batch over a batch of
synthetic device requests, commit / rollback included).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
                    [--shape llama8b] [--batch 16] [--layers L] [--greedy] [--weight-bits 8|4]
                    [--workload step|accept|attention|serve]

Prints ONE JSON line.  Metric: verified (committed) tokens per second at the Llama-3-8B shape.
`value` is measured with the draft distributions already in device memory, `e2e` with them in
pinned host memory (copied in and results copied out inside the timed region).  Drafts come from
distributions correlated with the target's own logits (`--drafts independent`: from distributions
that ignore the target).  `roofline` is for the tensor-core linear-layer kernel, the dominant one;
`kernel_ms` splits an untouched step by kind of kernel from per-launch device timestamps,
`kernel_ms_serialised` is the same with events between the kernels.  `independent_drafts` / `greedy` time the same
step with drafts that ignore the target / with greedy verification.  `sweep` repeats the step at
other batch sizes (fewer steps, no end-to-end leg), `weights_8bit` / `weights_4bit` with the linear layers'
weights as e4m3 bytes / e2m1 nibbles (`--weight-bits 8` / `4` runs everything that way).  `--impl reference` times the CPU oracle.
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
# the 129 launches of a step; profiles/ncu_linear_layer_kernel_llama8b_2layer_b{16,64}.txt), keyed by
# (shape, layers, batch).  Only valid for the kernel source it was taken from: reported as null when that file has
# changed since.
TRAFFIC_LINEAR = {"bytes_per_launch": {("llama8b", 32, 16): 117.9e6, ("llama8b", 32, 64): 125.4e6},
                  "source_sha1": "cdfa62a9961ce0a6bd7c9e43e29192ce2b26602f"}

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
    ap.add_argument("--workload", default="step", choices=["step", "accept", "attention", "serve"],
                    help="step: the full verification step (the headline); accept / attention: one kernel alone "
                         "on the acceptance-only / attention-only workload; serve: the server loop (queue, batch "
                         "planner, step) driven by a simulated population of devices")
    ap.add_argument("--devices", default="16,64,256,1024", help="serve: device counts to simulate")
    ap.add_argument("--draft-rate", type=float, default=5.24, help="serve: tokens per second a device drafts")
    ap.add_argument("--c-th", type=float, default=0.4, help="serve: confidence threshold of dynamic drafting")
    ap.add_argument("--policy", default="continuous", choices=["continuous", "static"])
    ap.add_argument("--static-batch", type=int, default=16, help="serve: batch size static batching waits for")
    ap.add_argument("--rounds", type=int, default=6, help="serve: verification rounds per device that are simulated")
    ap.add_argument("--max-batch", type=int, default=128, help="serve: most requests per step")
    ap.add_argument("--tau", type=float, default=1.0)
    ap.add_argument("--drafts", default="correlated", choices=["correlated", "independent"],
                    help="correlated: draft distributions built from the target's own logits (rho = 0.8), "
                         "independent: softmax of N(0,1) logits")
    ap.add_argument("--weight-bits", type=int, default=16, choices=[16, 8, 4],
                    help="8: the linear layers' weights as e4m3 bytes with one scale per output row (step workload)")
    ap.add_argument("--attention-impl", type=int, default=0, choices=[0, 1],
                    help="0: warp-level tensor-core attention kernel (default), 1: the tcgen05 kernel (head_dim 128)")
    ap.add_argument("--sweep", default="1,8,32,64,128", help="other batch sizes measured after the headline one")
    ap.add_argument("--no-sweep", action="store_true")
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


WEIGHT_BITS = 16   # --weight-bits 8 / 4: e4m3 bytes / e2m1 nibbles + one fp32 scale per output row


def linear_bytes(shape, T: int) -> float:
    """Bytes the linear layers must move in one step: every weight once (bf16, or a byte and the rows' scales),
    their bf16 inputs, their fp32 outputs."""
    es = 2 if shape.weight_dtype == "bf16" else 4
    if WEIGHT_BITS in (8, 4):
        return float(sum(n * k * WEIGHT_BITS // 8 + n * 4 + T * k * es + T * n * 4 for n, k in linear_shapes(shape)))
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
def _oracle_model(shape, weights_host):
    from oracle import oracle as O
    conv = lambda t: t.numpy() if t.dtype == torch.float32 else t
    w = {k: [conv(t) for t in v] if isinstance(v, list) else conv(v) for k, v in weights_host.items()}
    return O, O.OracleModel(shape, w)


def oracle_request(O, orc, shape, ks, ctx, seed, which: int, greedy: bool, drafts: str):
    """Loads request `which` of the batch into the oracle, builds its drafts (untimed) and times its verification.
    Correlated drafts are made from the oracle's own logits, position by position, with the generator the GPU arm
    uses on its logits.  Returns (seconds, committed tokens)."""
    K, V = I.make_kv(shape, ctx[which], seed, which)
    orc.load_kv(which, K.float().numpy(), V.float().numpy(), pending=1)
    del K, V
    k = ks[which]
    if drafts == "independent":
        d, q = I.make_drafts(shape.vocab, k, seed, which)
        d, q = d.numpy(), q.numpy()
    else:
        c = orc.ctx[which]
        d, q, tok = np.zeros(k, np.int32), np.zeros((k, shape.vocab), np.float32), c.pending
        for j in range(k):
            z = orc.forward_token(c, int(tok), c.n_kv + j)
            tok, qj = I.correlated_draft(torch.from_numpy(z), seed, which, j)
            d[j], q[j] = tok, qj.numpy()
    t0 = time.perf_counter()
    st, n_acc, nxt, _, _ = orc.verify(which, d, None if greedy else q, seed, 1.0, greedy)
    dt = time.perf_counter() - t0
    orc.release(which)
    return dt, n_acc + 1


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    shape, ks, ctx, seed = workload(args, 0)
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    w = I.weights_to(I.make_weights(shape, seed, device=dev), "cpu")
    O, orc = _oracle_model(shape, w)
    which = int(np.argmin(ks))
    times, toks = [], 0
    for i in range(args.warmup + args.steps):
        dt, n_tok = oracle_request(O, orc, shape, ks, ctx, seed, which, args.greedy, args.drafts)
        if i >= args.warmup:
            times.append(dt)
            toks += n_tok
    total = sum(times)
    value = toks / total
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "impl": "reference",
            "config": {"workload": workload_name(args, shape, ks, ctx)},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle",
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


def load_peaks():
    try:
        return json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json"))), "measured"
    except Exception:
        return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}, "fallback"


class Point:
    """One batch size of the step workload on its own engine: contexts with synthetic cache content, per-request
    drafts (correlated with the target, or independent), and the timing loops."""

    def __init__(self, B, args, shape, w_dev, batch, rank, local_rank, world, stream):
        self.B, self.args, self.shape, self.Bn, self.world, self.stream = B, args, shape, batch, world, stream
        sub = argparse.Namespace(**{**vars(args), "batch": batch})
        _, self.ks, self.ctx, self.seed = workload(sub, rank)
        self.name = workload_name(sub, shape, self.ks, self.ctx)
        self.T = sum(k + 1 for k in self.ks)
        self.dev = f"cuda:{local_rank}"
        n_pages = sum((c + k + 1 + 15) // 16 for c, k in zip(self.ctx, self.ks)) + 64
        self.eng = B.Engine(shape, w_dev, n_pages=n_pages, max_batch=batch, max_k=max(self.ks),
                            max_step_tokens=max(self.T, 16), temperature=1.0, greedy=args.greedy,
                            device_index=local_rank, stream=stream.cuda_stream, attention_impl=args.attention_impl,
                            linear_weight_bits=args.weight_bits)
        self.eng.shuffle_pages(self.seed)
        for i in range(batch):
            K, V = I.make_kv(shape, self.ctx[i], self.seed, i, device=self.dev)
            self.eng.load_kv(i, K, V, pending=1)
            del K, V
        self.res = (B.SledResult * batch)()
        self.lib = B.lib()
        self.ctx_ids = np.arange(batch, dtype=np.uint64)
        self.ctx_len = np.asarray(self.ctx, dtype=np.int64)
        self.pend = np.ones(batch, dtype=np.int32)

    # -- drafts
    def independent_drafts(self):
        d_host, q_dev = [], []
        for i in range(self.Bn):
            d, q = I.make_drafts(self.shape.vocab, self.ks[i], self.seed, i, device=self.dev)
            d_host.append(np.ascontiguousarray(d.cpu().numpy()))
            q_dev.append(q)
        return d_host, q_dev

    def correlated_drafts(self):
        """Draft j+1 of a request is drawn from a distribution built from the target's own logits at that position:
        k_max untimed greedy passes without commit over the drafts drawn so far, logits copied out after each."""
        eng, Bn, ks, V = self.eng, self.Bn, self.ks, self.shape.vocab
        eng.set_sampling(1.0, True)
        eng.set_commit(False)
        d_host = [np.zeros(k, np.int32) for k in ks]
        q_dev = [torch.zeros(k, V, device=self.dev) for k in ks]
        for j in range(max(ks)):
            have = [min(j, k) for k in ks]
            reqs = (self.B.SledRequest * Bn)()
            for i in range(Bn):
                reqs[i].ctx_id, reqs[i].k = i, have[i]
                reqs[i].draft_tokens = d_host[i].ctypes.data if have[i] else None
            rc = eng.verify_batch_raw(reqs, Bn, 0, self.res)
            if rc != 0:
                raise SystemExit(f"draft construction pass failed: {self.B.strerror(rc)}")
            n_rows = sum(h + 1 for h in have)
            logits = torch.empty(n_rows, V, device=self.dev)
            rc = self.lib.sled_debug_copy_logits(eng.h, logits.data_ptr(), n_rows)
            if rc != 0:
                raise SystemExit("sled_debug_copy_logits failed")
            row = 0
            for i in range(Bn):
                if ks[i] > j:
                    d, q = I.correlated_draft(logits[row + j], self.seed, i, j)
                    d_host[i][j] = d
                    q_dev[i][j] = q
                row += have[i] + 1
            del logits
        eng.set_sampling(1.0, self.args.greedy)
        eng.set_commit(True)
        return d_host, q_dev

    def marshal(self, d_host, qs):
        reqs = (self.B.SledRequest * self.Bn)()
        for i in range(self.Bn):
            reqs[i].ctx_id = i
            reqs[i].draft_tokens = d_host[i].ctypes.data if self.ks[i] else None
            reqs[i].draft_probs = None if (self.args.greedy or not self.ks[i]) else qs[i].data_ptr()
            reqs[i].k = self.ks[i]
        self._keep = (d_host, qs)
        return reqs

    # -- steps
    def one_step(self, reqs, step_seed):
        rc = self.eng.verify_batch_raw(reqs, self.Bn, step_seed, self.res)
        if rc != 0:
            raise SystemExit(f"sled_verify_batch failed: {self.B.strerror(rc)}")
        committed = 0
        for i in range(self.Bn):
            if self.res[i].status != 0:
                raise SystemExit(f"request {i} came back with status {self.res[i].status}")
            committed += self.res[i].n_accepted + 1
        # every context back to where it was (host bookkeeping only), so that all steps do the same work
        rc = self.lib.sled_debug_truncate_batch(self.eng.h, self.ctx_ids.ctypes.data, self.ctx_len.ctypes.data,
                                                self.pend.ctypes.data, self.Bn)
        if rc != 0:
            raise SystemExit("sled_debug_truncate_batch failed")
        return committed

    def timed(self, reqs, steps, warmup):
        for s in range(warmup):
            self.one_step(reqs, 100 + s)
        launches0 = self.eng.stats().kernels_launched
        if self.world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        committed = 0
        e0.record(self.stream)
        for s in range(steps):
            committed += self.one_step(reqs, 1000 + s)
        e1.record(self.stream)
        torch.cuda.synchronize()
        if self.world > 1:
            torch.distributed.barrier()
        return committed, e0.elapsed_time(e1), self.eng.stats().kernels_launched - launches0

    def kernel_times(self, reqs, mode, steps=5):
        """Device time by kind of kernel in extra steps: mode 1 = per-launch timestamps (launches overlap as in the
        timed steps), mode 2 = events between kernel groups (serialises them)."""
        self.eng.set_timing(mode)
        rows, n_rej = [], 0
        for s in range(steps):
            self.one_step(reqs, 2000 + s)
            st = self.eng.stats()
            rows.append((st.ms_linear, st.ms_attention, st.ms_accept, st.ms_other, st.ms_idle, st.ms_step))
            n_rej = sum(1 for i in range(self.Bn) if self.res[i].n_accepted < self.ks[i])
        self.eng.set_timing(0)
        med = [statistics.median(c) for c in zip(*rows)]
        names = ("linear", "attention", "accept", "other", "idle", "step")
        return dict(zip(names, med)), self.eng.stats().linear_launches_last_step, n_rej

    def summary(self, committed, ms, steps, n_rej, peaks):
        """Whole-step figures of one timed run (this rank)."""
        sb = step_bytes(self.shape, self.ks, self.ctx, n_rej)
        step_s = ms / steps / 1e3
        return {"ms_per_step": ms / steps, "tokens_per_s": committed / (ms / 1e3),
                "scored_positions_per_s": self.T / step_s,
                "acceptance_rate": (committed / steps - self.Bn) / max(sum(self.ks), 1),
                "step_bytes": sb, "frac_of_hbm_peak": sb / step_s / 1e9 / peaks["hbm_gbs"]}

    def linear_roofline(self, km, n_lin, peaks, peak_src):
        lb, lf = linear_bytes(self.shape, self.T), linear_flops(self.shape, self.T)
        lin = km["linear"]
        hbm, tc_s, tc_b = peaks["hbm_gbs"], peaks.get("bf16_tflops_sustained", 1400.0), peaks.get("bf16_tflops", 1590.0)
        if lb / (hbm * 1e9) >= lf / (tc_s * 1e12):
            ach = lb / (lin / 1e3) / 1e9
            roof = {"bound": "hbm", "achieved": ach, "peak": hbm, "unit": "GB/s", "frac": ach / hbm}
        else:
            ach = lf / (lin / 1e3) / 1e12
            roof = {"bound": "tensor", "achieved": ach, "peak": tc_s, "unit": "TFLOP/s", "frac": ach / tc_s,
                    "frac_of_burst_peak": ach / tc_b, "peak_kind": "sustained (the kernel runs inside a long step)"}
        roof.update({"kernel": "linear-layer kernel (all linear layers of a step)", "peak_source": peak_src,
                     "launches_per_step": n_lin, "avg_launch_ms": lin / max(n_lin, 1),
                     "algorithmic_bytes_per_launch": lb / max(n_lin, 1), "algorithmic_bytes_per_step": lb,
                     "algorithmic_flops_per_step": lf,
                     "time_basis": "per-launch device timestamps inside untouched steps: a launch is charged the time "
                                   "by which it extends the step beyond all earlier launches"})
        return roof

    def e2e_with_bf16_rows(self, d_host, q_dev, w_dev, local_rank, stream):
        """End-to-end steps on an engine that takes its draft rows in bf16 from pinned host memory.  Replaces this
        point's engine (one copy of the weights at a time)."""
        B, args = self.B, self.args
        n_pages = sum((c + k + 1 + 15) // 16 for c, k in zip(self.ctx, self.ks)) + 64
        self.eng.shutdown()
        torch.cuda.empty_cache()
        self.eng = B.Engine(self.shape, w_dev, n_pages=n_pages, max_batch=self.Bn, max_k=max(self.ks),
                            max_step_tokens=max(self.T, 16), temperature=1.0, greedy=False, device_index=local_rank,
                            stream=stream.cuda_stream, draft_probs_dtype="bf16", attention_impl=args.attention_impl,
                            linear_weight_bits=args.weight_bits)
        self.eng.shuffle_pages(self.seed)
        for i in range(self.Bn):
            K, V = I.make_kv(self.shape, self.ctx[i], self.seed, i, device=self.dev)
            self.eng.load_kv(i, K, V, pending=1)
            del K, V
        q16 = [q.to(torch.bfloat16).cpu().pin_memory() for q in q_dev]
        reqs = self.marshal(d_host, q16)
        n_steps = max(5, args.steps // 2)
        c, ms, _ = self.timed(reqs, n_steps, 3)
        return {"value": c / (ms / 1e3), "ms_per_step": ms / n_steps,
                "h2d_bytes_per_step": sum(k * self.shape.vocab * 2 for k in self.ks) + 64 * self.T}

    def close(self):
        self.eng.shutdown()
        torch.cuda.empty_cache()


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
    dev = f"cuda:{local_rank}"
    peaks, peak_src = load_peaks()
    w = I.make_weights(shape, seed, device=dev)
    global WEIGHT_BITS
    if args.weight_bits in (8, 4):
        WEIGHT_BITS = args.weight_bits
        args.no_cpu_baseline = True          # the oracle arm is timed on the 16-bit workload
        w, _ = I.quantize_linear_weights(w, dequantised=False, bits=args.weight_bits)
        torch.cuda.empty_cache()
    need_host_w = (rank == 0 and world == 1 and not args.no_cpu_baseline)
    w_host = I.weights_to(w, "cpu") if need_host_w else None
    stream = torch.cuda.Stream(device=dev)
    correlated = args.drafts == "correlated" and not args.greedy

    # ---- the headline point
    pt = Point(B, args, shape, w, args.batch, rank, local_rank, world, stream)
    Bn, T = pt.Bn, pt.T
    d_host, q_dev = pt.correlated_drafts() if correlated else pt.independent_drafts()
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    sampler.start()
    reqs_dev = pt.marshal(d_host, q_dev)
    committed, ms, launches = pt.timed(reqs_dev, args.steps, args.warmup)
    tok_all, ms_all = aggregate(float(committed), ms, world)
    value = tok_all / (ms_all / 1e3)

    e2e = None
    if not args.no_e2e:
        q_host = [q.cpu().pin_memory() for q in q_dev]
        reqs_host = pt.marshal(d_host, q_host)
        c2, ms2, _ = pt.timed(reqs_host, args.steps, args.warmup)
        t2, m2 = aggregate(float(c2), ms2, world)
        h2d = 0 if args.greedy else sum(k * shape.vocab * 4 for k in pt.ks)
        e2e = {"value": t2 / (m2 / 1e3), "unit": UNIT, "h2d_bytes_per_step": h2d + 64 * T,
               "d2h_bytes_per_step": 16 + 12 * Bn, "ms_per_step": m2 / args.steps}
        reqs_dev = pt.marshal(d_host, q_dev)
        del q_host
    clocks = sampler.stop()   # sampled over the warm-up and timed steps of both measurements

    km, n_lin, n_rej = pt.kernel_times(reqs_dev, 1)
    km_serial, _, _ = pt.kernel_times(reqs_dev, 2, steps=3)
    roof = pt.linear_roofline(km, n_lin, peaks, peak_src)
    traffic = None
    try:
        import hashlib
        src = open(os.path.join(ROOT, "paper_2506_09397_b200", "csrc", "gemm_tc.cu"), "rb").read()
        if hashlib.sha1(src).hexdigest() == TRAFFIC_LINEAR["source_sha1"]:
            traffic = TRAFFIC_LINEAR["bytes_per_launch"].get((shape.name, shape.n_layers, Bn))
    except Exception:
        pass
    roof["traffic"] = traffic
    head = pt.summary(committed, ms, args.steps, n_rej, peaks)
    step_s = ms_all / args.steps / 1e3
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_all / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": ({8: "bf16 (e4m3 weights)", 4: "bf16 (e2m1 weights)"}.get(args.weight_bits, "bf16")) if shape.weight_dtype == "bf16" else "f32",
            "data": "synthetic",
            "config": {"workload": pt.name, "tokens_scored_per_step": T,
                       "attention_kernel": "tcgen05" if args.attention_impl == 1 else "warp-level mma",
                       "linear_weight_bits": args.weight_bits,
                       "l2": "inputs larger than L2 (a step streams %.2f GB of weights)" % (args.weight_bits / 8 * 1e-9 * shape.streamed_params()),
                       "draft_distributions": ("target-correlated: draft logits = 0.8 z + 0.6 std(z) noise, z the target's "
                                               "own logits at that position (untimed passes), q = softmax, d ~ q"
                                               if correlated else "independent of the target (softmax of N(0,1) logits)"),
                       "kv": "synthetic N(0,1) cache content in permuted 16-token pages"},
            "clocks": clocks, "gpu_launches": int(launches),
            "scored_positions_per_s": T * world / step_s,
            "acceptance_rate": head["acceptance_rate"],
            "step_hbm": {"algorithmic_bytes": head["step_bytes"], "achieved_GBps": head["step_bytes"] / step_s / 1e9,
                         "frac_of_hbm_peak": head["step_bytes"] / step_s / 1e9 / peaks["hbm_gbs"], "peak_source": peak_src},
            "kernel_ms": km, "kernel_ms_serialised": km_serial, "roofline": roof}
    if e2e:
        line["e2e"] = e2e
    if correlated and not args.no_sweep:
        # the same step with drafts that ignore the target (acceptance is then low: nearly every request stops at its
        # first draft), as a second figure
        d2, q2 = pt.independent_drafts()
        r2 = pt.marshal(d2, q2)
        c_i, ms_i, _ = pt.timed(r2, max(5, args.steps // 2), 3)
        s_i = pt.summary(c_i, ms_i, max(5, args.steps // 2), Bn, peaks)
        line["independent_drafts"] = {k: s_i[k] for k in ("ms_per_step", "tokens_per_s", "acceptance_rate", "frac_of_hbm_peak")}
        del d2, q2, r2
        # greedy verification of the headline's drafts (argmax comparison: the draft rows are not read)
        pt.eng.set_sampling(1.0, True)
        c_g, ms_g, _ = pt.timed(reqs_dev, max(5, args.steps // 2), 3)
        s_g = pt.summary(c_g, ms_g, max(5, args.steps // 2), 0, peaks)
        line["greedy"] = {k: s_g[k] for k in ("ms_per_step", "tokens_per_s", "acceptance_rate", "frac_of_hbm_peak")}
        pt.eng.set_sampling(1.0, False)
    if e2e and not args.greedy and not args.no_sweep:
        # the same end-to-end step with the draft rows sent as bf16 (half the bytes; decisions then use the rounded
        # rows); it replaces the point's engine, so it comes last
        line["e2e"]["bf16_rows"] = pt.e2e_with_bf16_rows(d_host, q_dev, w, local_rank, stream)
    del d_host, q_dev, reqs_dev
    pt.close()

    # ---- other batch sizes of the same workload (fewer steps; no end-to-end leg)
    sweep = []
    if not args.no_sweep and world == 1:
        for b in [int(x) for x in args.sweep.split(",") if x]:
            if b == args.batch:
                continue
            sp = Point(B, args, shape, w, b, rank, local_rank, world, stream)
            dh, qd = sp.correlated_drafts() if correlated else sp.independent_drafts()
            torch.cuda.synchronize()
            smp = ClockSampler(local_rank)
            smp.start()
            rq = sp.marshal(dh, qd)
            n_steps = max(5, args.steps // 2)
            c_s, ms_s, _ = sp.timed(rq, n_steps, 3)
            clk = smp.stop()
            km_s, n_lin_s, n_rej_s = sp.kernel_times(rq, 1, steps=3)
            entry = {"batch": b, "tokens_scored_per_step": sp.T, "steps": n_steps, "workload": sp.name}
            entry.update(sp.summary(c_s, ms_s, n_steps, n_rej_s, peaks))
            entry["kernel_ms"] = km_s
            r = sp.linear_roofline(km_s, n_lin_s, peaks, peak_src)
            entry["linear_layers"] = {k: r[k] for k in ("bound", "achieved", "peak", "unit", "frac") if k in r}
            lf = linear_flops(shape, sp.T)
            tf = lf / (km_s["linear"] / 1e3) / 1e12
            entry["linear_layers"].update({"tflops": tf, "frac_of_sustained_bf16_peak": tf / peaks.get("bf16_tflops_sustained", 1400.0),
                                           "frac_of_burst_bf16_peak": tf / peaks.get("bf16_tflops", 1590.0)})
            entry["clocks"] = clk
            sweep.append(entry)
            del dh, qd, rq
            sp.close()
        line["sweep"] = sweep

    # ---- the same step with 8-bit and 4-bit weights in the linear layers (the paper sweeps 16-, 8- and 4-bit precision)
    if not args.no_sweep and world == 1 and args.weight_bits == 16 and shape.weight_dtype == "bf16":
        for bits, key, fmt in ((8, "weights_8bit", "e4m3 bytes"), (4, "weights_4bit", "e2m1 nibbles, two to a byte,")):
            wn, _ = I.quantize_linear_weights(w, dequantised=False, bits=bits)
            argsn = argparse.Namespace(**{**vars(args), "weight_bits": bits})
            WEIGHT_BITS = bits
            rows = []
            for b in sorted({args.batch, 1}, reverse=True):
                sp = Point(B, argsn, shape, wn, b, rank, local_rank, world, stream)
                dh, qd = sp.correlated_drafts() if correlated else sp.independent_drafts()
                torch.cuda.synchronize()
                rq = sp.marshal(dh, qd)
                n_steps = max(5, args.steps // 2)
                c_s, ms_s, _ = sp.timed(rq, n_steps, 3)
                km_s, n_lin_s, n_rej_s = sp.kernel_times(rq, 1, steps=3)
                entry = {"batch": b, "tokens_scored_per_step": sp.T, "steps": n_steps, "workload": sp.name}
                entry.update(sp.summary(c_s, ms_s, n_steps, n_rej_s, peaks))
                entry["kernel_ms"] = km_s
                r = sp.linear_roofline(km_s, n_lin_s, peaks, peak_src)
                entry["linear_layers"] = {k: r[k] for k in ("bound", "achieved", "peak", "unit", "frac") if k in r}
                rows.append(entry)
                del dh, qd, rq
                sp.close()
            WEIGHT_BITS = 16
            line[key] = {"format": fmt + " + one fp32 scale per output row; fp8 MMAs on activations split into two e4m3 "
                                         "parts; bytes counted with %d bits per weight" % bits, "points": rows}
            del wn
            torch.cuda.empty_cache()
    del w
    torch.cuda.empty_cache()

    if need_host_w:
        O, orc = _oracle_model(shape, w_host)
        t_all, tok_all_cpu = 0.0, 0
        for i in range(Bn):
            dt, n_tok = oracle_request(O, orc, shape, ks, ctx, seed, i, args.greedy, args.drafts)
            t_all += dt
            tok_all_cpu += n_tok
        line["cpu_baseline"] = {"value": tok_all_cpu / t_all, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle",
                                "seconds": t_all,
                                "sample": f"the whole batch of {Bn} requests, one after the other, one pass "
                                          "(drafts rebuilt from the oracle's own logits by the same generator, untimed)"}
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()


def _peaks():
    return load_peaks()


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
                   max_step_tokens=sum(qlens), attention_impl=args.attention_impl)
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


def run_serve(args):
    """The server loop under a simulated population of devices (Section 4 of the paper models verification requests
    the same way): every device is an independent source whose time to draft its next request is exponentially
    distributed with mean k / draft_rate; k follows dynamic drafting (Section 3.3): a device keeps drafting while
    the confidence of its newest token (uniform here, a stand-in) is at least c_th, up to max_k.  A device has one
    request outstanding at a time.  The server's clock advances by the measured device time of each sled_step;
    between steps it is idle until the next request arrives.  Reported per device count: whole-system token
    generation rate (committed tokens per simulated second), tokens per second and device, batch sizes, server
    utilisation; capacity = the largest simulated device count whose per-device rate is still at least 90 % of a
    lone device's."""
    import heapq
    from paper_2506_09397_b200 import binding as B
    shape = I.SHAPES[args.shape]
    if args.layers:
        shape = replace(shape, n_layers=args.layers)
    dev = "cuda:0"
    torch.cuda.set_device(0)
    counts = [int(x) for x in args.devices.split(",") if x]
    max_k, V = 8, shape.vocab
    w = I.make_weights(shape, args.seed, device=dev)
    if args.weight_bits in (8, 4):
        w, _ = I.quantize_linear_weights(w, dequantised=False, bits=args.weight_bits)
    stream = torch.cuda.Stream(device=dev)
    n_max = max(counts)
    ctx_len = I.draw_context_lengths(n_max, 128, 512, args.seed)
    # small populations are simulated for longer, so that every population answers a few hundred requests
    rounds_for = lambda n: max(args.rounds, -(-300 // n))
    n_pages = max(sum((c + 4 * rounds_for(n) * (max_k + 1) + 16 + 15) // 16 for c in ctx_len[:n]) for n in counts) + 64
    max_batch = min(args.max_batch, n_max)
    eng = B.Engine(shape, w, n_pages=n_pages, max_batch=max_batch, max_k=max_k, max_step_tokens=max_batch * (max_k + 1),
                   temperature=1.0, greedy=False, device_index=0, stream=stream.cuda_stream, probs_on_device=True,
                   linear_weight_bits=args.weight_bits)
    del w
    eng.server_config(B.SLED_BATCH_STATIC if args.policy == "static" else B.SLED_BATCH_CONTINUOUS,
                      min(args.static_batch, max_batch))
    # a pool of draft-distribution rows on the device; a request takes the first k rows of one pool entry
    pool = [I.make_drafts(V, max_k, args.seed, 7000 + i, device=dev)[1] for i in range(32)]
    torch.cuda.synchronize()
    rng = np.random.default_rng(args.seed)
    gen = torch.Generator(device=dev)
    gen.manual_seed(args.seed)
    mean_k = sum(k * (1 - args.c_th) ** (k - 1) * (args.c_th if k < max_k else 1.0) for k in range(1, max_k + 1))
    out = []
    for n_dev in sorted(counts):
        t_end = rounds_for(n_dev) * (mean_k / args.draft_rate + 0.005)   # about that many verification cycles of a lone device
        t_warm = 0.25 * t_end
        max_rounds = 4 * rounds_for(n_dev)                               # bounds how far a context can grow
        for i in range(n_dev):                                   # fresh contexts for every device count
            K, Vv = I.make_kv(shape, ctx_len[i], args.seed, i, device=dev)
            eng.load_kv(i, K, Vv, pending=1)
            del K, Vv
        # every launch shape once before the clock starts (first uses configure kernels)
        eng.set_commit(False)
        for b in sorted({1, min(3, n_dev), min(12, n_dev), min(20, n_dev), min(60, n_dev), min(max_batch, n_dev)}):
            tk = [eng.submit(i, np.zeros(max_k, np.int32), pool[0]) for i in range(b)]
            eng.step(0, flush=True)
            for x in tk:
                eng.poll(x)
        eng.set_commit(True)

        def draw_k():
            k = 1
            while k < max_k and rng.random() >= args.c_th:        # confident: draft another token
                k += 1
            return k

        heap = []
        for i in range(n_dev):
            k = draw_k()
            heapq.heappush(heap, (rng.exponential(k / args.draft_rate), i, k))
        t, busy, steps, tokens, served, latency, batch_sizes = 0.0, 0.0, 0, 0, 0, [], []
        rounds_done = {i: 0 for i in range(n_dev)}
        in_flight = {}
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        while t < t_end and (heap or in_flight):
            while heap and heap[0][0] <= t:                      # requests that have arrived by now
                ta, i, k = heapq.heappop(heap)
                q = pool[int(rng.integers(0, len(pool)))][:k]
                d = torch.multinomial(q, 1, generator=gen).reshape(k).to(torch.int32).cpu().numpy()
                in_flight[eng.submit(i, d, q)] = (i, ta, k, q)
            if not in_flight:
                t = heap[0][0]                                   # idle until the next arrival
                continue
            e0.record(stream)
            n = eng.step(1000 + steps, flush=not heap)          # static batching: flush when nobody else can come
            e1.record(stream)
            e1.synchronize()
            if n == 0:                                           # static batching still waiting for its batch
                t = heap[0][0]
                continue
            dt = e0.elapsed_time(e1) / 1e3
            t += dt
            steps += 1
            counted = t > t_warm
            if counted:
                busy += dt
                batch_sizes.append(n)
            for ticket in list(in_flight):
                r = eng.poll(ticket)
                if r is None:
                    continue
                i, ta, k, _ = in_flight.pop(ticket)
                if r[2] != 0:
                    raise SystemExit(f"request of device {i} failed with status {r[2]}")
                if counted:
                    tokens += r[0] + 1
                    served += 1
                    latency.append(t - ta)
                rounds_done[i] += 1
                if rounds_done[i] < max_rounds:
                    k2 = draw_k()
                    heapq.heappush(heap, (t + rng.exponential(k2 / args.draft_rate), i, k2))
        while in_flight:                                         # drain what is still queued (not counted)
            eng.step(0, flush=True)
            for ticket in list(in_flight):
                if eng.poll(ticket) is not None:
                    in_flight.pop(ticket)
        span = max(t, t_end) - t_warm
        entry = {"devices": n_dev, "wstgr_tokens_per_s": tokens / span, "tokens_per_s_per_device": tokens / span / n_dev,
                 "requests": served, "steps": len(batch_sizes), "mean_batch": float(np.mean(batch_sizes)) if batch_sizes else 0.0,
                 "max_batch_seen": int(max(batch_sizes)) if batch_sizes else 0, "server_utilisation": busy / span,
                 "mean_step_ms": 1e3 * busy / max(1, len(batch_sizes)),
                 "mean_response_ms": 1e3 * float(np.mean(latency)) if latency else None,
                 "measured_seconds": span, "tokens_per_request": tokens / max(1, served)}
        out.append(entry)
        for i in range(n_dev):
            eng.release(i)
    lone_rate = out[0]["tokens_per_s_per_device"]                # the smallest population: its requests hardly ever wait
    ok = [e["devices"] for e in out if e["tokens_per_s_per_device"] >= 0.9 * lone_rate]
    print(json.dumps({"metric": "wstgr_tokens_per_s", "value": max(e["wstgr_tokens_per_s"] for e in out), "unit": "tokens/s",
                      "n_gpus": 1, "higher_is_better": True, "dtype": "bf16" if shape.weight_dtype == "bf16" else "f32",
                      "data": "synthetic",
                      "config": {"workload": f"server loop, {shape.name} ({shape.n_layers} layers), {args.policy} batching, "
                                             f"devices drafting {args.draft_rate} tokens/s, c_th={args.c_th}, max_k={max_k}, "
                                             f"contexts 128..512, about {args.rounds} verification rounds per device simulated "
                                             "(more for small populations; the first quarter of the time is not counted)",
                                 "draft_distributions": "independent of the target (softmax of N(0,1) logits)",
                                 "linear_weight_bits": args.weight_bits},
                      "capacity_devices": {"value": max(ok) if ok else 0, "rule": "largest simulated count whose devices still get >= 90 % of "
                                           "the token rate of the smallest population's", "reached_largest_simulated": bool(ok) and max(ok) == max(counts)},
                      "by_devices": out}))
    eng.shutdown()


def main(argv=None):
    args = parse_args(argv)
    if args.impl == "reference":
        run_reference(args)
    elif args.workload == "serve":
        run_serve(args)
    elif args.workload == "accept":
        run_accept_only(args)
    elif args.workload == "attention":
        run_attention_only(args)
    else:
        run_sled(args)


if __name__ == "__main__":
    main()
