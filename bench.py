"""Benchmark of the speculative-decoding hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--batch B] [--gamma G] [--impl reference]
    python bench.py --profile-pass --model NAME [--layers L] [--batch B] [--rows R] [--context C]   (profiler driver)

Prints ONE JSON line (rank 0).  For N > 1 it is launched with torchrun, one
process per GPU; ranks are independent replicas (the path has no exchange
step), timed between barriers, max over ranks.

Workloads (--workload)
  llama7b   (default) Llama-7B-shaped bf16 target with a 160M-shaped draft, random
            init, 1024-token prompts, batch --batch (1), gamma --gamma (2), T = 1.
            A step is one iteration of Algorithm 1 for the whole batch: gamma
            draft passes, one target pass over gamma+1 rows, speculative sampling,
            commit and KV roll-back.
  t5xxl     T5-XXL-shaped bf16 encoder-decoder target with a T5-small-shaped draft,
            512-token sources (encoders run once, in the prompt pass), 128 decoded
            tokens, gamma --gamma (5).
  gpt97m    the paper-shaped GPT-like 97M target with its 6M draft, 8k vocabulary.
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
    top_k, top_p = 0, 1.0  # Section 2.2's truncations, off in the headline workload (--top-k / --top-p)

    def description(self):
        cut = {"top_k": self.top_k, "top_p": self.top_p} if (self.top_k or self.top_p != 1.0) else {}
        return {"workload": self.name, "batch": self.batch, "gamma": self.gamma, "vocab": self.vocab,
                "temperature": self.temperature, "draft_noise": list(self.noises), **cut,
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
            xs = binding.spec_sample(ql_d.view(-1, self.vocab), torch.from_numpy(draw).to(device), self.temperature,
                                     top_k=self.top_k, top_p=self.top_p)
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
        self.binding.spec_verify_sample(tl, ql, xs, us, self.temperature, self.n, self.t, self.ws,
                                        top_k=self.top_k, top_p=self.top_p)
        # kernels of this library launched: statistics pass + finishing pass (+ one selection pass per active cut)
        return 2 + (0 < self.top_k < self.vocab) + (0.0 < self.top_p < 1.0)

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
        self.binding.spec_verify_sample(tl, ql, xs, us, self.temperature, self.n, self.t, self.ws,
                                        top_k=self.top_k, top_p=self.top_p)
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
        while time.perf_counter() - t0 < budget_s or done < 2:
            b = done % self.batch
            for i in range(self.gamma):
                xs[b, i] = oracle_sampling.sample_token(ql[b, i], draw[b * self.gamma + i], self.temperature,
                                                        self.top_k, self.top_p)[0]
            res = oracle_sampling.verify_step(tl[b], ql[b], xs[b], us[b], self.temperature, 1.0, self.top_k, self.top_p)
            tokens += res.n_accepted + 1
            done += 1
        dt = time.perf_counter() - t0
        return tokens / dt, f"{done} sequences drawn from one batch of {self.batch} (draft draws + verify), {dt:.1f} s"


# --------------------------------------------------------------------------- #
# workload: speculative decoding of a model pair (Algorithm 1, device-resident loop)
# --------------------------------------------------------------------------- #
def gpu_weights(cfg, seed, device):
    """Seeded random-init weights drawn on the GPU with torch's generator (matrices
    N(0, 0.02^2), head N(0, head_std^2), gains 1; bf16 models stored as bf16)."""
    import torch
    from paper_2211_17192_b200 import workloads
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    out = {}
    for name, shape, kind in workloads.tensor_shapes(cfg):
        if kind == "gain":
            out[name] = torch.ones(shape, device=device)
            continue
        std = cfg["head_std"] if kind == "head" else cfg["bias_std"] if kind == "bias" else workloads.INIT_STD
        t = torch.randn(shape, device=device, generator=g, dtype=torch.float32) * std
        out[name] = t.to(torch.bfloat16) if cfg["dtype"] == "bf16" and kind != "bias" else t
    return out


def decode_stream(name):
    """Whether a tensor is streamed by a decoder pass (encoder-decoder models: not the
    encoder stack, nor the projections of the encoder output, which run once per source)."""
    return not (name.startswith("enc.") or name.endswith(("wkv_x", "rel_bias")))


def weight_stream_bytes(cfg):
    """Bytes of one pass over the model: every block matrix and the LM head once."""
    from paper_2211_17192_b200 import workloads
    elem = 2 if cfg["dtype"] == "bf16" else 4
    if cfg["arch"] == "bigram":
        return cfg["vocab"] * elem  # one row of the table
    total = 0
    for name, shape, kind in workloads.tensor_shapes(cfg):
        if kind == "gain" or name in ("pos_emb",) or (name == "tok_emb" and not cfg["tied"]) or not decode_stream(name):
            continue
        total += int(np.prod(shape)) * elem
    return total


class GenerationWorkload:
    dtype = "bf16"

    def __init__(self, name, target, draft, batch, prompt_len, n_new, gamma, temperature=1.0, layers=None):
        from paper_2211_17192_b200 import workloads
        self.name, self.target_name, self.draft_name = name, target, draft
        self.layers = layers
        self.tcfg, self.dcfg = workloads.model_config(target), workloads.model_config(draft)  # (prepare applies --layers)
        self.batch, self.prompt_len, self.n_new, self.gamma, self.temperature = batch, prompt_len, n_new, gamma, temperature
        self.adaptive_gamma_max = 0  # set from the command line

    def description(self):
        return {"workload": self.name, "target": self.target_name, "draft": self.draft_name, "batch": self.batch,
                "prompt_len": self.prompt_len, "n_new": self.n_new, "gamma": self.gamma,
                "temperature": self.temperature, "kv_dtype": "fp16" if self.tcfg["dtype"] == "bf16" else "fp32",
                **({"target_layers_override": self.layers} if self.layers else {}),
                "l2": "one pass streams the target's weights (>> 126 MB L2) from HBM",
                "parallelism": "replicas"}

    def prepare(self, rank, device, iterations, weights=None):
        """`weights`: (target, draft) tensors of another workload on the same pair of shapes (not drawn again)."""
        import torch
        from paper_2211_17192_b200 import binding, workloads
        self.torch, self.binding, self.device = torch, binding, device
        self.tcfg = workloads.model_config(self.target_name)
        if self.layers:
            self.tcfg = workloads.scaled_config(self.tcfg, n_layers=self.layers)
        self.dcfg = workloads.model_config(self.draft_name)
        self.dtype = "bf16" if self.tcfg["dtype"] == "bf16" else "f32"
        self.tw, self.dw = weights if weights else (gpu_weights(self.tcfg, 100 + rank, device), gpu_weights(self.dcfg, 200 + rank, device))
        grow = max(self.n_new, iterations * (self.gamma + 1) + 64)
        top_gamma = max(self.gamma, self.adaptive_gamma_max, 1)
        self.max_len = self.prompt_len + grow + top_gamma + 2
        self.engine = binding.Engine(self.tcfg, self.tw, self.dcfg, self.dw, max_batch=self.batch, max_len=self.max_len,
                                     page_size=64, max_gamma=top_gamma)
        self.prompts = [workloads.make_prompt(1000 * rank + b, self.prompt_len, self.tcfg["vocab"]) for b in range(self.batch)]
        self.budget_tokens = grow
        self.kv_elem_bytes = 2 if self.engine.kv_dtype in ("fp16", "bf16") else 4

    def close(self):
        self.engine.close()
        self.engine = None

    def kv_bytes(self, context):
        """K,V bytes one target pass reads: the cached rows of every sequence, in the cache's element type."""
        c = self.tcfg
        return self.batch * context * 2 * c["n_layers"] * c["n_kv_heads"] * c["d_head"] * self.kv_elem_bytes

    def launches_per_iteration(self):
        # per block: 4 GEMMs, 2 norms, RoPE/append, attention, activation (+ the combine kernel when the
        # key slices are not merged inside a cluster: long contexts); embed, final norm, head, its reduction
        long_context = self.prompt_len > 256
        fwd = lambda cfg, combine: 1 + (9 + combine) * cfg["n_layers"] + 3
        draft = 1 if self.dcfg["arch"] in ("bigram", "copy") else fwd(self.dcfg, 0)  # (few slices: merged in the cluster)
        target = fwd(self.tcfg, 1 if long_context else 0)
        return 1 + self.gamma * (1 + draft + 1) + 1 + target + 2 + 1

    def timed_decode(self, warmup, steps, gamma):
        """Device time of `steps` iterations after `warmup` untimed ones (prompt pass untimed)."""
        self.engine.begin(self.prompts, self.budget_tokens, gamma, self.temperature, 7)
        _, before = self.engine.step(warmup)
        _, after = self.engine.step(steps)
        tokens = after["tokens"] - before["tokens"]
        stats = {k: after[k] - before[k] for k in ("iterations", "tokens", "tests_evaluated", "tests_passed")}
        return tokens, after["decode_ms"], stats

    def e2e(self, calls):
        """The public call with host buffers: prompts in, tokens out, prompt pass included."""
        t0 = time.perf_counter()
        tokens = 0
        for i in range(calls):
            out, _ = self.engine.generate(self.prompts, self.n_new, self.gamma, self.temperature, 11 + i)
            tokens += out.size
        return tokens, time.perf_counter() - t0

    def e2e_bytes(self):
        return self.batch * self.prompt_len * 4 + self.batch * 4, self.batch * self.n_new * 4

    def adaptive(self, gamma_max):
        """Section 3.5: gamma picked by the library burst by burst; decode time only, like `timed_decode`."""
        self.engine.generate_adaptive(self.prompts, self.n_new, gamma_max, self.temperature, 7)  # captures the graphs
        out, st, trace = self.engine.generate_adaptive(self.prompts, self.n_new, gamma_max, self.temperature, 7)
        used = {}
        for g, n in trace:
            used[g] = used.get(g, 0) + n
        return {"gamma_max": gamma_max, "tokens_per_s": out.size / (st["decode_ms"] / 1e3),
                "iterations_by_gamma": {str(g): used[g] for g in sorted(used)},
                "alpha": st["tests_passed"] / max(1, st["tests_evaluated"]),
                "note": "spec_generate_adaptive over n_new tokens: two calibration bursts (gamma 1 and gamma_max), then "
                        "the gamma that maximises Eq. 1 over a line fitted to the measured iteration times"}

    def pass_times(self, repeats=20):
        """Device time of single passes (graph-replayed, events on the library's stream):
        the target on 1 and on gamma+1 rows, the draft on 1 row, at the prompt's context length."""
        eng, torch = self.engine, self.torch
        tok = np.stack([p[: self.prompt_len - 1] for p in self.prompts])
        def timed(which, rows):
            return eng.time_forward(which, self.batch, rows, repeats)
        eng.reset()
        chunk = max(1, 64 // self.batch)  # the teacher-forced entry point takes 64 rows per call
        stateless = self.dcfg["arch"] in ("bigram", "copy")  # no cache to fill (a copy draft has no teacher-forced pass)
        for which in ((0,) if stateless else (0, 1)):
            for c0 in range(0, tok.shape[1], chunk):
                eng.forward_logits(which, tok[:, c0:c0 + chunk])
        self.pass_context = self.prompt_len - 1
        return {"target_1row_ms": timed(0, 1), "target_rows_ms": timed(0, self.gamma + 1), "draft_1row_ms": timed(1, 1)}

    def gemm_roofline(self, rows):
        """The weight-streaming GEMM kernel alone, as the engine launches it: every block
        matrix and the head of the target (decoder) once at `rows` rows, tile-major
        weights, activations split once per inner dimension beforehand, split-K partial
        sums left in the workspace.  The sweep (one GEMM launch per matrix, nothing else)
        is captured in a CUDA graph and timed with events on its stream."""
        torch, binding = self.torch, self.binding
        mats = [(n, t) for n, t in self.tw.items() if t.dim() == 2 and n not in ("tok_emb", "pos_emb") and decode_stream(n)]
        if self.tcfg["tied"]:
            mats.append(("head", self.tw["tok_emb"]))
        stream = torch.cuda.Stream(self.device)
        with torch.cuda.stream(stream):
            packed = {n: binding.spec_pack_weight(t) for n, t in mats}
            ks = sorted({t.shape[1] for _, t in mats})
            ws, xs = {}, {}
            for k in ks:
                need = max(binding.spec_linear_workspace_bytes(rows, t.shape[0], k) for _, t in mats if t.shape[1] == k)
                ws[k] = torch.empty(need, dtype=torch.uint8, device=self.device)
                xs[k] = torch.randn(rows, k, device=self.device)
                first, first_t = next((n, t) for n, t in mats if t.shape[1] == k)
                binding.spec_linear_partials(xs[k], packed[first], first_t.shape[0], ws[k])  # leaves the split of x
            def sweep():
                for n, t in mats:
                    binding.spec_linear_partials(None, packed[n], t.shape[0], ws[t.shape[1]], split_input=False,
                                                 rows=rows, k=t.shape[1])
            sweep()
            stream.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                sweep()
            graph.replay()
            stream.synchronize()
            samples = []
            for _ in range(7):  # the median of several replays, each timed on its own
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                graph.replay()
                b.record(stream)
                stream.synchronize()
                samples.append(a.elapsed_time(b))
        nbytes = sum(t.numel() * t.element_size() for _, t in mats)
        ms = statistics.median(samples)
        del packed
        torch.cuda.empty_cache()
        return nbytes, ms, len(mats)

    def cpu_sample(self, budget_s):
        """The oracle on a bounded sample: both models at full width and reduced depth
        (2 layers each), a short prompt, a few iterations; extrapolated to the full
        depth by streamed weight bytes."""
        from oracle import generate as oracle_generate
        from oracle.decoder import Decoder
        from paper_2211_17192_b200 import workloads
        small_t = workloads.scaled_config(self.tcfg, n_layers=min(2, self.tcfg["n_layers"]))
        small_d = self.dcfg if self.dcfg["arch"] in ("bigram", "copy") else workloads.scaled_config(self.dcfg, n_layers=min(2, self.dcfg["n_layers"]))
        dtype = np.float32 if self.tcfg["d_model"] >= 2048 else np.float64
        if not hasattr(self, "_cpu_models"):  # built once, outside every timed sample
            if self.dcfg["arch"] == "bigram":
                from oracle.ngram import BigramTable
                draft_model = BigramTable(workloads.make_weights(self.dcfg, 2)["table"], dtype=np.float32)
            elif self.dcfg["arch"] == "copy":
                from oracle.ngram import CopyFromContext
                draft_model = CopyFromContext(self.dcfg["vocab"], self.dcfg["ngram"])
            else:
                draft_model = Decoder(small_d, workloads.make_weights(small_d, 2), dtype=dtype)
            self._cpu_models = (Decoder(small_t, workloads.make_weights(small_t, 1), dtype=dtype), draft_model)
        target, draft = self._cpu_models
        prompt = workloads.make_prompt(3, 32, self.tcfg["vocab"])
        t0 = time.perf_counter()
        tokens = iters = 0
        n_new = 4 * (self.gamma + 1)
        while time.perf_counter() - t0 < budget_s or iters == 0:
            res = oracle_generate.speculative_generate(target, draft, prompt, n_new, self.gamma, self.temperature, seed=iters)
            tokens += len(res.tokens)
            iters += len(res.iterations)
        dt = time.perf_counter() - t0
        full = weight_stream_bytes(self.tcfg) + self.gamma * weight_stream_bytes(self.dcfg)
        small = weight_stream_bytes(small_t) + self.gamma * weight_stream_bytes(small_d)
        value = tokens / dt * small / full
        sample = (f"{iters} iterations of Algorithm 1, batch 1, 32-token prompt, both models at full width and "
                  f"{small_t['n_layers']}+{small_d.get('n_layers', 0)} layers in {np.dtype(dtype).name}, {dt:.1f} s; "
                  f"scaled by streamed weight bytes ({small / full:.3f}) to the full depth")
        return value, sample


class EncDecWorkload(GenerationWorkload):
    """Encoder-decoder pair: `prompt_len` is the source length; the encoders run once
    per source (inside the prompt pass, untimed in `value`, timed in `e2e`) and the
    decoders start from the start token."""

    def description(self):
        d = super().description()
        d["source_len"] = d.pop("prompt_len")
        d["l2"] = "one pass streams the target decoder's weights (>> 126 MB L2) from HBM"
        return d

    def prepare(self, rank, device, iterations, weights=None):
        import torch
        from paper_2211_17192_b200 import binding, workloads
        self.torch, self.binding, self.device = torch, binding, device
        self.tcfg = workloads.model_config(self.target_name)
        if self.layers:
            self.tcfg = workloads.scaled_config(self.tcfg, n_layers=self.layers, n_enc_layers=self.layers)
        self.dcfg = workloads.model_config(self.draft_name)
        self.dtype = "bf16"
        self.tw = gpu_weights(self.tcfg, 100 + rank, device)
        self.dw = gpu_weights(self.dcfg, 200 + rank, device)
        grow = max(self.n_new, iterations * (self.gamma + 1) + 64)
        top_gamma = max(self.gamma, self.adaptive_gamma_max, 1)
        self.max_len = 1 + grow + top_gamma + 2
        self.engine = binding.Engine(self.tcfg, self.tw, self.dcfg, self.dw, max_batch=self.batch, max_len=self.max_len,
                                     page_size=64, max_gamma=top_gamma, max_src_len=self.prompt_len)
        self.prompts = [workloads.make_prompt(1000 * rank + b, self.prompt_len, self.tcfg["vocab"]) for b in range(self.batch)]
        self.budget_tokens = grow
        self.kv_elem_bytes = 2 if self.engine.kv_dtype in ("fp16", "bf16") else 4

    def launches_per_iteration(self):
        # per decoder block: 7 GEMMs, 3 norms, K/V append, cross-attention queries, 2 attentions, activation
        fwd = lambda cfg: 1 + 15 * cfg["n_layers"] + 3
        return 1 + self.gamma * (1 + fwd(self.dcfg) + 1) + 1 + fwd(self.tcfg) + 2 + 1

    def kv_bytes(self, context):
        c = self.tcfg
        per_position = 2 * c["n_layers"] * c["n_kv_heads"] * c["d_head"] * self.kv_elem_bytes
        return self.batch * (context + self.prompt_len) * per_position  # self-attention rows + cross-attention rows

    def pass_times(self, repeats=20):
        """Device time of single passes (graph-replayed) at a decoder context of
        n_new / 2 tokens: the target on 1 and gamma+1 rows, the draft on 1 row."""
        eng = self.engine
        context = max(1, self.n_new // 2)
        self.pass_context = context
        def timed(which, rows):
            return eng.time_forward(which, self.batch, rows, repeats)
        eng.encode(self.prompts)
        for which in (0, 1):
            for c0 in range(0, context, 32):
                eng.forward_logits(which, np.zeros((self.batch, min(32, context - c0)), dtype=np.int32))
        return {"target_1row_ms": timed(0, 1), "target_rows_ms": timed(0, self.gamma + 1), "draft_1row_ms": timed(1, 1)}

    def cpu_sample(self, budget_s):
        """The oracle on a bounded sample: both models at full width with one encoder and
        one decoder block each, a 32-token source; extrapolated to the full decoder depth
        by streamed weight bytes."""
        from oracle import generate as oracle_generate
        from oracle.encdec import START_TOKEN, EncoderDecoder
        from paper_2211_17192_b200 import workloads
        small_t = workloads.scaled_config(self.tcfg, n_layers=1, n_enc_layers=1)
        small_d = workloads.scaled_config(self.dcfg, n_layers=1, n_enc_layers=1)
        if not hasattr(self, "_cpu_models"):  # built and encoded once, outside every timed sample
            target = EncoderDecoder(small_t, workloads.make_weights(small_t, 1), dtype=np.float32)
            draft = EncoderDecoder(small_d, workloads.make_weights(small_d, 2), dtype=np.float32)
            source = workloads.make_prompt(3, 32, self.tcfg["vocab"])
            target.encode(source)
            draft.encode(source)
            self._cpu_models = (target, draft)
        target, draft = self._cpu_models
        t0 = time.perf_counter()
        tokens = iters = 0
        n_new = self.gamma + 1
        while time.perf_counter() - t0 < budget_s or iters == 0:
            res = oracle_generate.speculative_generate(target, draft, [START_TOKEN], n_new, self.gamma, self.temperature, seed=iters)
            tokens += len(res.tokens)
            iters += len(res.iterations)
        dt = time.perf_counter() - t0
        full = weight_stream_bytes(self.tcfg) + self.gamma * weight_stream_bytes(self.dcfg)
        small = weight_stream_bytes(small_t) + self.gamma * weight_stream_bytes(small_d)
        value = tokens / dt * small / full
        sample = (f"{iters} iterations of Algorithm 1 (decode only, encoders run before the clock), batch 1, 32-token "
                  f"source, both models at full width and 1 decoder layer in float32, {dt:.1f} s; scaled by "
                  f"streamed weight bytes ({small / full:.3f}) to the full depth")
        return value, sample


def make_workload(args):
    wl = _make_workload(args)
    wl.adaptive_gamma_max = args.adaptive_gamma_max
    return wl


def _make_workload(args):
    if args.workload == "sampler":
        wl = SamplerWorkload()
        wl.top_k, wl.top_p = args.top_k, args.top_p
        if wl.top_k or wl.top_p != 1.0:
            wl.name += f"_k{wl.top_k}_p{wl.top_p:g}"
        return wl
    batch = args.batch or 1
    if args.workload == "t5xxl":
        gamma = args.gamma or 5
        return EncDecWorkload(f"t5xxl_small_b{batch}_g{gamma}", "t5xxl_target", "t5small_draft", batch,
                              args.prompt_len or 512, 128, gamma, args.temperature, args.layers)
    if args.workload == "gpt97m":
        return GenerationWorkload("gpt97m_6m_b1", "gpt97m_target", "gpt6m_draft", batch, args.prompt_len or 128, 512,
                                  args.gamma or 5, args.temperature, args.layers)
    gamma = args.gamma or 2
    if args.draft == "bigram":  # a negligible-cost draft: one table row per step instead of a model pass
        return GenerationWorkload(f"llama7b_bigram_b{batch}_g{gamma}", "llama7b_target", "bigram_32k", batch,
                                  args.prompt_len or 1024, 256, gamma, args.temperature, args.layers)
    if args.draft == "copy":  # parameter-less: guesses copied from the context (Section 3.6)
        return GenerationWorkload(f"llama7b_copy_b{batch}_g{gamma}", "llama7b_target", "copy_32k", batch,
                                  args.prompt_len or 1024, 256, gamma, args.temperature, args.layers)
    return GenerationWorkload(f"llama7b_160m_b{batch}_g{gamma}", "llama7b_target", "llama160m_draft", batch,
                              args.prompt_len or 1024, 256, gamma, args.temperature, args.layers)


WORKLOAD_NAMES = ["llama7b", "t5xxl", "gpt97m", "sampler"]


# --------------------------------------------------------------------------- #
def load_tensor_peak():
    """Measured dense bf16 rate of a library GEMM timed alone (burst), TFLOP/s; the earlier measurement if the file is absent."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["bf16_tflops"]), "measured"
    return 1590.0, "fallback"


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


def aggregate_over_ranks(dist, device, times, counts):
    """Replicas only: every rank ran the same job on its own sequences.  The job's time
    is the slowest rank's (MAX), its work the sum over ranks (SUM); no other exchange."""
    import torch
    t = torch.tensor(list(times), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    c = torch.tensor(list(counts), dtype=torch.int64, device=device)
    dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return [float(v) for v in t], [int(v) for v in c]


def run_reference(args, wl):
    """The reference arm: the CPU oracle as it stands, on the machine's host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    values = []
    sample = ""
    per_step = max(0.5, min(60.0 / max(1, args.steps + args.warmup), 4.0 * args.cpu_budget))  # about a minute in all by default
    for _ in range(args.warmup):
        wl.cpu_sample(per_step)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        v, sample = wl.cpu_sample(per_step)
        values.append(v)
    dt = time.perf_counter() - t0
    value = statistics.mean(values)
    out = {
        "impl": "reference", "metric": "generated tokens/s", "value": value, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1000.0 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32" if getattr(wl, "tcfg", {}).get("d_model", 0) >= 2048 else "f64",  # what the oracle computes in here
        "data": "synthetic",
        "config": wl.description(),
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cpu_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out))


def run_sampler(args, wl, torch, device, local, barrier):
    """Timed region: K calls of spec_verify_sample captured in one CUDA graph."""
    wl.prepare(int(os.environ.get("RANK", "0")), device)
    stream = torch.cuda.Stream(device)
    with torch.cuda.stream(stream):
        for i in range(args.warmup):
            wl.step(i)
        stream.synchronize()
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
        elapsed_ms = start.elapsed_time(stop)
        t_end = time.time() + 0.5  # keep the GPU under this load while the clocks are sampled
        while time.time() < t_end:
            graph.replay()
        stream.synchronize()
        clock_info = clocks.stop(w0, time.time())
        tokens = wl.tokens_emitted(args.warmup, args.steps)
    for i in range(3):
        wl.e2e_step(i)
    barrier()
    e0 = time.perf_counter()
    e2e_tokens = 0
    for i in range(args.steps):
        e2e_tokens += wl.e2e_step(i)
    barrier()
    e2e_s = time.perf_counter() - e0
    peak, peak_kind = load_peaks()
    launch_s = elapsed_ms / args.steps / 1e3
    achieved = wl.algorithmic_bytes() / launch_s / 1e9
    extras = {
        "roofline": {"bound": "hbm", "kernel": "verify_stats_kernel+verify_finish_kernel", "achieved": achieved,
                     "peak": peak, "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                     "frac_of_nominal_8tbs": achieved / 8000.0, "traffic": 122.98e6,
                     "traffic_note": "dram bytes read per launch from the ncu capture under profiles/",
                     "algorithmic_bytes_per_launch": wl.algorithmic_bytes(), "launch_us": 1e6 * launch_s},
    }
    return dict(tokens=tokens, elapsed_ms=elapsed_ms, e2e_tokens=e2e_tokens, e2e_s=e2e_s, launches=launches,
                clocks=clock_info, extras=extras)


def measure_pair(wl, analysis, peak, warmup, steps):
    """Tokens/s, target-only tokens/s, acceptance, cost ratios and the target pass against the HBM
    roofline for one prepared generation workload."""
    tokens, ms, stats = wl.timed_decode(warmup, steps, wl.gamma)
    base_tokens, base_ms, _ = wl.timed_decode(warmup, steps, 0)  # target-only, same kernels
    times = wl.pass_times(10)
    alpha = stats["tests_passed"] / max(1, stats["tests_evaluated"])
    tpi = stats["tokens"] / max(1, stats["iterations"])
    pass_bytes = weight_stream_bytes(wl.tcfg) + wl.kv_bytes(wl.pass_context)
    gbs = pass_bytes / (times["target_rows_ms"] / 1e3) / 1e9
    return {"workload": wl.name, "batch": wl.batch, "gamma": wl.gamma, "iterations": steps,
            "tokens_per_s": tokens / (ms / 1e3), "target_only_tokens_per_s": base_tokens / (base_ms / 1e3),
            "speedup_vs_target_only": (tokens / ms) / (base_tokens / base_ms), "alpha": alpha,
            "c": times["draft_1row_ms"] / times["target_1row_ms"], "kappa": times["target_rows_ms"] / times["target_1row_ms"],
            "generalised_closed_form": analysis.generalised_speedup(tpi, times["target_1row_ms"], times["target_rows_ms"],
                                                                    times["draft_1row_ms"], wl.gamma),
            "pass_ms": times, "verify_pass": {"bytes": pass_bytes, "gbs": gbs, "frac": gbs / peak}}


def sampler_point(torch, device):
    """The standalone sampler workload (batch 64 x 8 positions x vocabulary 32000) in the same run:
    microseconds per call (CUDA graph of 60 calls over three rotating input sets, events) and the
    fraction of the measured HBM rate."""
    wl = SamplerWorkload()
    wl.prepare(0, device)
    stream = torch.cuda.Stream(device)
    with torch.cuda.stream(stream):
        for i in range(3):
            wl.step(i)
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for i in range(60):
                wl.step(i)
        graph.replay()
        stream.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        graph.replay()
        b.record(stream)
        stream.synchronize()
    us = 1e3 * a.elapsed_time(b) / 60
    peak, kind = load_peaks()
    gbs = wl.algorithmic_bytes() / (us / 1e6) / 1e9
    return {"workload": wl.name, "us_per_call": us, "gbs": gbs, "frac": gbs / peak, "peak_kind": f"of {kind}"}


def run_generation(args, wl, torch, device, local, barrier):
    """Timed region: K iterations of Algorithm 1 (gamma draft passes, one target pass
    over gamma+1 rows, speculative sampling, commit and roll-back), replayed as a
    CUDA graph per iteration by the library and timed with events on its stream."""
    from oracle import analysis  # closed forms only, for the report (rank 0)
    rank = int(os.environ.get("RANK", "0"))
    long_steps = max(200, args.steps)  # (also measured: a stretch long enough for the acceptance rate to settle)
    # ... as far as the model's positions reach: every iteration may add gamma + 1 tokens to the context
    context0 = 1 if isinstance(wl, EncDecWorkload) else wl.prompt_len
    from paper_2211_17192_b200 import workloads
    room = workloads.model_config(wl.target_name)["max_positions"] - context0 - 64 - wl.gamma - 3
    long_steps = max(args.steps, min(long_steps, room // (wl.gamma + 1) - args.warmup))
    wl.prepare(rank, device, args.warmup + long_steps)
    clocks = ClockSampler(local)
    clocks.start()
    time.sleep(0.15)
    barrier()
    w0 = time.time()
    tokens, elapsed_ms, stats = wl.timed_decode(args.warmup, args.steps, wl.gamma)
    barrier()
    clock_info = clocks.stop(w0, time.time())
    base_tokens, base_ms, _ = wl.timed_decode(args.warmup, args.steps, 0)  # target-only, same kernels
    for _ in range(1):
        wl.e2e(1)
    barrier()
    e2e_tokens, e2e_s = wl.e2e(3)
    barrier()
    extras = {}
    if rank == 0:
        peak, peak_kind = load_peaks()
        rows = wl.batch * (wl.gamma + 1)
        nbytes, gemm_ms, n_mats = wl.gemm_roofline(rows)
        achieved = nbytes / (gemm_ms / 1e3) / 1e9
        times = wl.pass_times()
        alpha = stats["tests_passed"] / max(1, stats["tests_evaluated"])
        tok_per_iter = stats["tokens"] / max(1, stats["iterations"])
        c = times["draft_1row_ms"] / times["target_1row_ms"]
        # Timing only: the accept decision replaced by Bernoulli(alpha*) from the same
        # uniforms, so that the speedup can be set against the closed forms across the
        # paper's range of alpha (a random-init pair sits at one uncontrolled alpha).
        sweep = []
        base_rate = base_tokens / base_ms
        for imposed in (0.5, 0.6, 0.7, 0.8, 0.9):
            wl.engine.set_imposed_acceptance(imposed)
            s_tokens, s_ms, s_stats = wl.timed_decode(3, min(args.steps, 40), wl.gamma)
            s_tpi = s_stats["tokens"] / max(1, s_stats["iterations"])
            sweep.append({"alpha": imposed, "tokens_per_s": s_tokens / (s_ms / 1e3),
                          "speedup_vs_target_only": (s_tokens / s_ms) / base_rate,
                          "measured_alpha": s_stats["tests_passed"] / max(1, s_stats["tests_evaluated"]),
                          "theorem_3_8": analysis.walltime_improvement(imposed, wl.gamma, c),
                          "generalised": analysis.generalised_speedup(s_tpi, times["target_1row_ms"], times["target_rows_ms"],
                                                                      times["draft_1row_ms"], wl.gamma)})
        wl.engine.set_imposed_acceptance(None)
        kv_bytes = wl.kv_bytes(wl.pass_context)
        pass_bytes = weight_stream_bytes(wl.tcfg) + kv_bytes
        pass_gbs = pass_bytes / (times["target_rows_ms"] / 1e3) / 1e9
        # DRAM bytes of one pass from the ncu capture of a 2-block cut of the 7B-shaped target (batch 1, 3 rows, 1024 cached
        # tokens): 363.7 MB per block (354.4 MB of weights), 266.8 MB for the head, embedding and final norm; traffic grows in
        # proportion to the blocks.  Only for the workload that capture is of.
        pass_traffic, pass_traffic_note = None, "no capture for this workload"
        if args.workload == "llama7b" and wl.batch == 1 and wl.gamma == 2 and not args.layers:
            pass_traffic = wl.tcfg["n_layers"] * 363.7e6 + 266.8e6
            pass_traffic_note = ("dram__bytes_read.sum + dram__bytes_write.sum of every kernel of a pass, captured on a 2-block "
                                 "cut and scaled by the block count (profiles/ncu_pass_traffic_llama7b_rows3_ctx1024.txt)")
        long_tokens, long_ms, long_stats = wl.timed_decode(args.warmup, long_steps, wl.gamma)
        # the other configurations of the scope, measured in this same run (short: 30 iterations each)
        others = []
        if args.workload == "llama7b" and args.configs and not args.layers:
            for batch, gamma in ((16, 4), (32, 6)):
                other = GenerationWorkload(f"llama7b_160m_b{batch}_g{gamma}", wl.target_name, wl.draft_name, batch, wl.prompt_len,
                                           wl.n_new, gamma, wl.temperature)
                other.prepare(rank, device, 3 + 30, weights=(wl.tw, wl.dw))
                others.append(measure_pair(other, analysis, peak, 3, 30))
                other.close()
            wl.close()
            del wl.tw, wl.dw
            torch.cuda.empty_cache()
            for other in (GenerationWorkload("gpt97m_6m_b1", "gpt97m_target", "gpt6m_draft", 1, 128, 512, 5, wl.temperature),
                          EncDecWorkload("t5xxl_small_b1_g5", "t5xxl_target", "t5small_draft", 1, 512, 128, 5, wl.temperature)):
                other.prepare(rank, device, 3 + 30)
                others.append(measure_pair(other, analysis, peak, 3, 30))
                other.close()
                del other.tw, other.dw
                torch.cuda.empty_cache()
            others.append(sampler_point(torch, device))
        extras = {
            "value_long": {"tokens_per_s": long_tokens / (long_ms / 1e3), "iterations": long_steps,
                           "alpha": long_stats["tests_passed"] / max(1, long_stats["tests_evaluated"])},
            "configs": others,
            "speedup_vs_target_only": (tokens / elapsed_ms) / (base_tokens / base_ms),
            "target_only_tokens_per_s": base_tokens / (base_ms / 1e3),
            "alpha": alpha, "tokens_per_iteration": tok_per_iter, "c": c,
            "kappa": times["target_rows_ms"] / times["target_1row_ms"],
            "closed_form": {"theorem_3_8": analysis.walltime_improvement(alpha, wl.gamma, c),
                            "expected_tokens_eq_1": analysis.expected_tokens(alpha, wl.gamma),
                            "generalised": analysis.generalised_speedup(tok_per_iter, times["target_1row_ms"],
                                                                        times["target_rows_ms"], times["draft_1row_ms"],
                                                                        wl.gamma)},
            "pass_ms": times,
            # Section 3.5: the gamma that maximises Theorem 3.8 for the measured alpha and c, and the one that
            # maximises the generalised form when every extra verified row costs what the measured kappa implies
            "best_gamma": {"theorem_3_8": analysis.best_gamma(alpha, c, 32) if 0.0 < alpha < 1.0 else None,
                           "generalised": max(range(1, 33), key=lambda g_: analysis.generalised_speedup(
                               analysis.expected_tokens(alpha, g_), times["target_1row_ms"],
                               times["target_1row_ms"] * (1.0 + (times["target_rows_ms"] / times["target_1row_ms"] - 1.0) * g_ / max(wl.gamma, 1)),
                               times["draft_1row_ms"], g_)) if 0.0 < alpha < 1.0 else None},
            "imposed_acceptance_sweep": sweep,
            **({"adaptive_gamma": wl.adaptive(wl.adaptive_gamma_max)} if wl.adaptive_gamma_max else {}),
            # the quantity the metric names: one target pass over gamma+1 rows, weights + the cached K,V rows it
            # reads, against the HBM copy rate (the whole pass: GEMM chain, attention and the small kernels between)
            "roofline": {"bound": "hbm", "kernel": "target pass over gamma+1 rows (gemm_tc_kernel chain, attention, small kernels)",
                         "achieved": pass_gbs, "peak": peak, "unit": "GB/s", "frac": pass_gbs / peak,
                         "peak_kind": f"of {peak_kind}", "frac_of_nominal_8tbs": pass_gbs / 8000.0,
                         "algorithmic_bytes_per_pass": pass_bytes, "weight_bytes": weight_stream_bytes(wl.tcfg),
                         "kv_bytes": kv_bytes, "ms_per_pass": times["target_rows_ms"],
                         "traffic": pass_traffic,
                         "traffic_note": pass_traffic_note,
                         "note": "weights + K,V rows of the context in the cache's element type (for encoder-decoders also "
                                 "the source rows), one pass over gamma+1 rows, graph replays timed with events on the "
                                 "library's stream",
                         "gemm_kernel": {
                         "kernel": "gemm_tc_kernel", "achieved": achieved, "frac": achieved / peak,
                         "frac_of_nominal_8tbs": achieved / 8000.0,
                         "algorithmic_bytes_per_launch": nbytes / n_mats,
                         # the same sweep against the tensor pipes: where rows approach the ridge (about 216-262 rows)
                         # the GEMMs stop being purely bandwidth-bound; two MMAs per k-step (split activations)
                         "tensor": (lambda tp: {"useful_tflops": rows * nbytes / (gemm_ms / 1e3) / 1e12,
                                                "issued_tflops": 2 * rows * nbytes / (gemm_ms / 1e3) / 1e12,
                                                "peak": tp[0], "peak_kind": f"of {tp[1]} (burst)",
                                                "frac_issued": 2 * rows * nbytes / (gemm_ms / 1e3) / 1e12 / tp[0],
                                                "note": "2 x rows x parameters flop per sweep; issued counts both "
                                                        "bf16 terms of the activations"})(load_tensor_peak()),
                         "launch_us": 1e3 * gemm_ms / n_mats,
                         "note": f"all {n_mats} weight matrices of the target once at {rows} rows through spec_linear_partials "
                                 "(the GEMM kernel alone, tile-major weights, one launch per matrix back to back), "
                                 "CUDA graph, median of 7 replays, events on its stream"}},
        }
    launches = wl.launches_per_iteration() * args.steps
    return dict(tokens=tokens, elapsed_ms=elapsed_ms, e2e_tokens=e2e_tokens, e2e_s=e2e_s, launches=launches,
                clocks=clock_info, extras=extras)


def profile_pass(args):
    """One forward-pass shape, repeated, for profilers (`--profile-pass`): builds the named model of
    `workloads.model_config` (optionally at reduced depth, full width; weights drawn on the GPU), feeds
    `--context` tokens per sequence through the teacher-forced entry point, and then replays one pass
    over `--rows` new rows per sequence `--repeats` times with `spec_time_forward`.  Every kernel of the
    decode path therefore appears in the launch list with exactly the shape it has in a verification pass
    (rows = gamma + 1) or a draft step (rows = 1), which is what `ncu -k regex:<kernel>` wants.  Prints
    the device time per pass."""
    import torch

    import __graft_entry__ as entry
    from paper_2211_17192_b200 import binding, workloads
    entry.build()
    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    cfg = workloads.model_config(args.model)
    if args.layers:
        cfg = workloads.scaled_config(cfg, n_layers=args.layers, n_enc_layers=min(cfg["n_enc_layers"], args.layers))
    t5 = cfg["arch"] == "t5"
    batch = args.batch or 1
    eng = binding.Engine(cfg, gpu_weights(cfg, 1, device), max_batch=batch, max_len=args.context + args.rows + 8,
                         page_size=64, max_gamma=max(args.rows - 1, 1), kv_dtype=args.kv_dtype,
                         max_src_len=args.source if t5 else 0, pass_kernel=args.pass_kernel)
    if t5:
        eng.encode([workloads.make_prompt(b, args.source, cfg["vocab"]) for b in range(batch)])
    tokens = np.stack([workloads.make_prompt(100 + b, args.context, cfg["vocab"]) for b in range(batch)])
    chunk = max(1, 64 // batch)
    for c0 in range(0, args.context, chunk):
        eng.forward_logits(0, tokens[:, c0:c0 + chunk])
    ms = eng.time_forward(0, batch, args.rows, args.repeats)
    print(json.dumps({"profile_pass": args.model, "layers": cfg["n_layers"], "batch": batch, "rows": args.rows,
                      "context": args.context, "kv_dtype": eng.kv_dtype, "pass_kernel": bool(args.pass_kernel),
                      "ms_per_pass": ms}))
    eng.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=6)
    ap.add_argument("--workload", default="llama7b", choices=WORKLOAD_NAMES)
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--gamma", type=int, default=None)
    ap.add_argument("--temperature", type=float, default=1.0)
    ap.add_argument("--prompt-len", type=int, default=None, help="override the workload's prompt length (profiling)")
    ap.add_argument("--draft", default="model", choices=["model", "bigram", "copy"],
                    help="llama7b workload: the 160M-shaped draft model, or a bigram table (negligible-cost draft)")
    ap.add_argument("--layers", type=int, default=None, help="override the target's depth, full width (profiling)")
    ap.add_argument("--top-k", type=int, default=0, help="sampler workload: top-k standardisation of both models")
    ap.add_argument("--top-p", type=float, default=1.0, help="sampler workload: nucleus standardisation of both models")
    ap.add_argument("--adaptive-gamma-max", type=int, default=0,
                    help="also report decoding with gamma chosen by the library burst by burst, up to this value")
    ap.add_argument("--no-configs", dest="configs", action="store_false",
                    help="llama7b workload: skip the other configurations (batch 16 and 32, GPT 97M/6M, T5-XXL/small, sampler)")
    ap.add_argument("--profile-pass", action="store_true",
                    help="profiler driver: replay one pass shape (--model --layers --batch --rows --context --repeats) and exit")
    ap.add_argument("--model", default="llama7b_target", help="--profile-pass: model name of workloads.model_config")
    ap.add_argument("--rows", type=int, default=3, help="--profile-pass: new rows per sequence in the timed pass")
    ap.add_argument("--context", type=int, default=1024, help="--profile-pass: cached tokens per sequence before the timed pass")
    ap.add_argument("--source", type=int, default=512, help="--profile-pass: source length (encoder-decoder models)")
    ap.add_argument("--repeats", type=int, default=3, help="--profile-pass: replays of the pass")
    ap.add_argument("--kv-dtype", default=None, choices=["fp32", "fp16", "bf16"], help="--profile-pass: cached K,V row type")
    ap.add_argument("--pass-kernel", action="store_true", help="--profile-pass: the persistent pass kernel instead of the kernel chain")
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--cpu-budget", type=float, default=15.0, help="seconds of oracle time for cpu_baseline")
    args = ap.parse_args()
    if args.profile_pass:
        profile_pass(args)
        return
    if args.steps is None:
        args.steps = 300 if args.workload == "sampler" else 100
    args.warmup = max(args.warmup, 3) if args.impl == "native" else args.warmup
    wl = make_workload(args)

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

    runner = run_sampler if args.workload == "sampler" else run_generation
    res = runner(args, wl, torch, device, local, barrier)
    tokens, elapsed_ms, e2e_tokens, e2e_s, launches = (res[k] for k in ("tokens", "elapsed_ms", "e2e_tokens", "e2e_s", "launches"))

    if world > 1:
        (elapsed_ms, e2e_s), (tokens, e2e_tokens, launches) = aggregate_over_ranks(
            dist, device, [elapsed_ms, e2e_s], [tokens, e2e_tokens, launches])

    if rank == 0:
        cpu_value, cpu_sample = wl.cpu_sample(args.cpu_budget) if world == 1 else (None, "skipped for N > 1")
        h2d, d2h = wl.e2e_bytes()
        out = {
            "metric": "generated tokens/s", "value": tokens / (elapsed_ms / 1000.0), "unit": "tokens/s",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": elapsed_ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype,
            "data": "synthetic", "config": wl.description(),
            "clocks": res["clocks"],
            "e2e": {"value": e2e_tokens / e2e_s, "unit": "tokens/s", "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h},
            "gpu_launches": launches,
        }
        out.update(res["extras"])
        out["cpu_baseline"] = {"value": cpu_value, "unit": "tokens/s", "cores": cpu_threads(), "kind": "oracle",
                               "sample": cpu_sample}
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
