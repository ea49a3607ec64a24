"""Benchmark of the speculative-decoding hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints ONE JSON line (rank 0).  For N > 1 it is launched with torchrun, one
process per GPU; ranks are independent replicas (the path has no exchange
step), timed between barriers, max over ranks.

Workloads
  sampler   the standalone speculative-sampling kernel: batch 64 x
            (gamma+1 = 8) x vocab 32000, T = 1, draft logits = target + N(0, s^2)
            with s rotating over {0.5, 1, 2}.  A step is one call of
            spec_verify_sample on one batch.
"""

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


# --------------------------------------------------------------------------- #
# clocks
# --------------------------------------------------------------------------- #
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [p.strip() for p in line.split(",")]))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.12)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        inside = [r for (t, r) in self.rows if t0 <= t <= t1 + 0.06] or [r for (_, r) in self.rows]
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in inside:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for name, val in zip(names, r[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------- #
# workload: standalone speculative-sampling kernel
# --------------------------------------------------------------------------- #
class SamplerWorkload:
    name = "sampler_b64_g7_v32000"
    batch, gamma, vocab, temperature = 64, 7, 32000, 1.0
    noises = (0.5, 1.0, 2.0)
    dtype = "f32"

    def description(self):
        return {"workload": self.name, "batch": self.batch, "gamma": self.gamma, "vocab": self.vocab,
                "temperature": self.temperature, "draft_noise": list(self.noises),
                "l2": "inputs rotate over 3 logit sets (369 MB) > 126 MB L2",
                "parallelism": "replicas"}

    # bytes the method must move per step: every p and q logit once, tokens, uniforms, outputs
    def algorithmic_bytes(self):
        b, g, v = self.batch, self.gamma, self.vocab
        return b * (2 * g + 1) * v * 4 + b * g * 4 + b * (g + 1) * 4 + b * 8

    def host_inputs(self, rank):
        from paper_2211_17192_b200 import workloads
        sets = []
        for k, s in enumerate(self.noises):
            tl, ql = workloads.make_sampler_logits(1000 * rank + k, self.batch, self.gamma, self.vocab, s)
            us = workloads.make_uniform_grid(2000 * rank + k, (self.batch, self.gamma + 1))
            draw = workloads.make_uniform_grid(3000 * rank + k, (self.batch * self.gamma,))
            sets.append((tl, ql, us, draw))
        return sets

    def prepare(self, rank, device):
        import torch
        from paper_2211_17192_b200 import binding
        self.binding = binding
        self.torch = torch
        self.device = device
        self.host = self.host_inputs(rank)
        self.dev_sets = []
        for tl, ql, us, draw in self.host:
            tl_d, ql_d = torch.from_numpy(tl).to(device), torch.from_numpy(ql).to(device)
            # x_i ~ q_i drawn by the library's own sampler (Algorithm 1's draft draws)
            xs = binding.spec_sample(ql_d.view(-1, self.vocab), torch.from_numpy(draw).to(device), self.temperature)
            self.dev_sets.append((tl_d, ql_d, xs.view(self.batch, self.gamma).contiguous(),
                                  torch.from_numpy(us).to(device)))
        self.n = torch.empty(self.batch, dtype=torch.int32, device=device)
        self.t = torch.empty(self.batch, dtype=torch.int32, device=device)
        need = binding.spec_verify_sample_workspace_bytes(self.batch, self.gamma, self.vocab)
        self.ws = torch.empty(need, dtype=torch.uint8, device=device)
        # pinned host copies for the end-to-end leg
        self.pinned = []
        for (tl, ql, us, _), (_, _, xs, _) in zip(self.host, self.dev_sets):
            self.pinned.append(tuple(torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
                                     for a in (tl, ql, xs.cpu().numpy(), us)))
        self.stage = tuple(torch.empty_like(a, device=device) for a in self.pinned[0])
        self.n_host = torch.empty(self.batch, dtype=torch.int32).pin_memory()
        self.t_host = torch.empty(self.batch, dtype=torch.int32).pin_memory()
        torch.cuda.synchronize()

    def step(self, i):
        tl, ql, xs, us = self.dev_sets[i % len(self.dev_sets)]
        self.binding.spec_verify_sample(tl, ql, xs, us, self.temperature, self.n, self.t, self.ws)
        return 2  # kernels of this library launched: statistics pass + finishing pass

    def tokens_emitted(self, first_step, steps):
        """Tokens the timed steps emitted (n accepted + 1 per sequence).  Each
        input set gives the same result every time, so this is counted after
        the timed region instead of inside it."""
        per_set = []
        for k in range(len(self.dev_sets)):
            self.step(k)
            per_set.append(int(self.n.sum().item()) + self.batch)
        return sum(per_set[(first_step + i) % len(per_set)] for i in range(steps))

    def e2e_step(self, i):
        """Host buffers in, host results out: copies are inside the timed region."""
        src = self.pinned[i % len(self.pinned)]
        for d, s in zip(self.stage, src):
            d.copy_(s, non_blocking=True)
        tl, ql, xs, us = self.stage
        self.binding.spec_verify_sample(tl, ql, xs, us, self.temperature, self.n, self.t, self.ws)
        self.n_host.copy_(self.n, non_blocking=True)
        self.t_host.copy_(self.t, non_blocking=True)
        self.torch.cuda.current_stream().synchronize()
        return int(self.n_host.sum()) + self.batch

    def e2e_bytes(self):
        h2d = sum(a.numel() * a.element_size() for a in self.pinned[0])
        return h2d, 2 * self.batch * 4

    # the oracle on a bounded sample of the same workload
    def cpu_sample(self, budget_s):
        from oracle import sampling as oracle_sampling
        tl, ql, us, draw = self.host[1] if hasattr(self, "host") else self.host_inputs(0)[1]
        xs = np.zeros((self.batch, self.gamma), dtype=np.int32)
        t0 = time.perf_counter()
        done = tokens = 0
        while done < self.batch and (time.perf_counter() - t0 < budget_s or done < 2):
            b = done
            for i in range(self.gamma):
                xs[b, i] = oracle_sampling.sample_token(ql[b, i], draw[b * self.gamma + i], self.temperature)[0]
            res = oracle_sampling.verify_step(tl[b], ql[b], xs[b], us[b], self.temperature)
            tokens += res.n_accepted + 1
            done += 1
        dt = time.perf_counter() - t0
        return tokens / dt, f"{done} of {self.batch} sequences of one batch (draft draws + verify), {dt:.1f} s"


WORKLOADS = {"sampler": SamplerWorkload}


# --------------------------------------------------------------------------- #
def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info()]
        return max(n) if n else 1
    except Exception:
        return 1


def run_reference(args, wl):
    """The reference arm: the CPU oracle as it stands, on the machine's host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    values = []
    sample = ""
    for _ in range(args.warmup):
        wl.cpu_sample(0.5)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        v, sample = wl.cpu_sample(max(1.0, 60.0 / max(1, args.steps)))
        values.append(v)
    dt = time.perf_counter() - t0
    value = statistics.mean(values)
    out = {
        "impl": "reference", "metric": "generated tokens/s", "value": value, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1000.0 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": wl.description(),
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=6)
    ap.add_argument("--workload", default="sampler", choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--cpu-budget", type=float, default=12.0, help="seconds of oracle time for cpu_baseline")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "native" else args.warmup
    wl = WORKLOADS[args.workload]()

    if args.impl == "reference":
        run_reference(args, wl)
        return

    import torch
    import torch.distributed as dist

    import __graft_entry__ as entry

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    if rank == 0:
        entry.build()
    if world > 1:
        dist.barrier()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    wl.prepare(rank, device)
    stream = torch.cuda.Stream(device)
    with torch.cuda.stream(stream):
        for i in range(args.warmup):
            wl.step(i)
        stream.synchronize()
        # The K timed steps are captured once in a CUDA graph so that the device
        # never waits for the Python launch loop; the timed region is one replay.
        graph = torch.cuda.CUDAGraph()
        launches = 0
        with torch.cuda.graph(graph, stream=stream):
            for i in range(args.steps):
                launches += wl.step(args.warmup + i)
        graph.replay()  # untimed: uploads the graph
        stream.synchronize()

        clocks = ClockSampler(local)
        clocks.start()
        time.sleep(0.15)
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        w0 = time.time()
        start.record(stream)
        graph.replay()
        stop.record(stream)
        barrier()
        w1 = time.time()
        elapsed_ms = start.elapsed_time(stop)
        # keep the clocks sampler busy long enough to see the GPU under this load
        t_end = time.time() + 0.5
        while time.time() < t_end:
            graph.replay()
        stream.synchronize()
        w1 = time.time()
        clock_info = clocks.stop(w0, w1)
        tokens = wl.tokens_emitted(args.warmup, args.steps)
    kernel_ms = [elapsed_ms / args.steps]

    # end-to-end leg: pinned host buffers in, host results out
    for i in range(3):
        wl.e2e_step(i)
    barrier()
    e0 = time.perf_counter()
    e2e_tokens = 0
    for i in range(args.steps):
        e2e_tokens += wl.e2e_step(i)
    barrier()
    e2e_s = time.perf_counter() - e0

    if world > 1:
        t = torch.tensor([elapsed_ms, e2e_s], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        elapsed_ms, e2e_s = float(t[0]), float(t[1])
        c = torch.tensor([tokens, e2e_tokens, launches], dtype=torch.int64, device=device)
        dist.all_reduce(c, op=dist.ReduceOp.SUM)
        tokens, e2e_tokens, launches = int(c[0]), int(c[1]), int(c[2])

    if rank == 0:
        peak, peak_kind = load_peaks()
        avg_kernel_s = statistics.mean(kernel_ms) / 1000.0
        achieved = wl.algorithmic_bytes() / avg_kernel_s / 1e9
        cpu_value, cpu_sample = wl.cpu_sample(args.cpu_budget) if world == 1 else (None, "skipped for N > 1")
        h2d, d2h = wl.e2e_bytes()
        out = {
            "metric": "generated tokens/s", "value": tokens / (elapsed_ms / 1000.0), "unit": "tokens/s",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": elapsed_ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype,
            "data": "synthetic", "config": wl.description(),
            "clocks": clock_info,
            "e2e": {"value": e2e_tokens / e2e_s, "unit": "tokens/s", "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h},
            "gpu_launches": launches,
            "roofline": {"bound": "hbm", "kernel": "verify_stats_kernel+verify_finish_kernel", "achieved": achieved,
                         "peak": peak,
                         "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                         "frac_of_nominal_8tbs": achieved / 8000.0, "traffic": None,
                         "algorithmic_bytes_per_launch": wl.algorithmic_bytes(),
                         "launch_us": 1e3 * statistics.mean(kernel_ms)},
            "cpu_baseline": {"value": cpu_value, "unit": "tokens/s", "cores": 1, "kind": "oracle",
                             "sample": cpu_sample},
        }
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
