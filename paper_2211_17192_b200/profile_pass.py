"""One forward-pass shape, repeated: a small driver for profilers.

    python -m paper_2211_17192_b200.profile_pass --model llama7b_target --layers 2 \
        --batch 8 --rows 3 --context 1024 [--repeats 3] [--kv-dtype fp32]

Builds the named model of `workloads.model_config` (optionally at reduced depth,
full width; weights drawn on the GPU), feeds `context` tokens per sequence
through the teacher-forced entry point, and then replays one pass over `rows`
new rows per sequence `repeats` times with `spec_time_forward`.  Every kernel
of the decode path therefore appears in the launch list with exactly the shape
it has in a verification pass (rows = gamma + 1) or a draft step (rows = 1),
which is what an `ncu -k regex:<kernel>` capture wants.  Prints the device time
per pass.
"""

import argparse

import numpy as np
import torch

from . import binding, workloads


def _gpu_weights(cfg, seed, device):
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    out = {}
    for name, shape, kind in workloads.tensor_shapes(cfg):
        if kind == "gain":
            out[name] = torch.ones(shape, device=device)
            continue
        std = cfg["head_std"] if kind == "head" else cfg["bias_std"] if kind == "bias" else workloads.INIT_STD
        t = torch.randn(shape, device=device, generator=g, dtype=torch.float32) * std
        out[name] = t.to(torch.bfloat16) if cfg["dtype"] == "bf16" and kind != "bias" else t
    return out


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--model", default="llama7b_target")
    ap.add_argument("--layers", type=int, default=None, help="reduced depth (full width)")
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--rows", type=int, default=3, help="new rows per sequence in the timed pass")
    ap.add_argument("--context", type=int, default=1024, help="cached tokens per sequence (decoder) before the timed pass")
    ap.add_argument("--source", type=int, default=512, help="source length (encoder-decoder models)")
    ap.add_argument("--repeats", type=int, default=3)
    ap.add_argument("--kv-dtype", default="fp32", choices=["fp32", "bf16"])
    args = ap.parse_args()

    from .build import build
    build()
    device = torch.device("cuda", 0)
    cfg = workloads.model_config(args.model)
    if args.layers:
        cfg = workloads.scaled_config(cfg, n_layers=args.layers, n_enc_layers=min(cfg["n_enc_layers"], args.layers))
    t5 = cfg["arch"] == "t5"
    eng = binding.Engine(cfg, _gpu_weights(cfg, 1, device), max_batch=args.batch, max_len=args.context + args.rows + 8,
                         page_size=64, max_gamma=max(args.rows - 1, 1), kv_dtype=args.kv_dtype,
                         max_src_len=args.source if t5 else 0)
    if t5:
        eng.encode([workloads.make_prompt(b, args.source, cfg["vocab"]) for b in range(args.batch)])
    tokens = np.stack([workloads.make_prompt(100 + b, args.context, cfg["vocab"]) for b in range(args.batch)])
    chunk = max(1, 64 // args.batch)
    for c0 in range(0, args.context, chunk):
        eng.forward_logits(0, tokens[:, c0:c0 + chunk])
    ms = eng.time_forward(0, args.batch, args.rows, args.repeats)
    print(f"{args.model} layers={cfg['n_layers']} batch={args.batch} rows={args.rows} context={args.context}: {ms:.4f} ms per pass")
    eng.close()


if __name__ == "__main__":
    main()
