"""A few forward passes of one named workload, for captures under a profiler.

    python -m paper_2312_07987_b200.profile_driver CONFIG [--passes N] [--batch B] [--flush]

Sets the layer up from the seeded synthetic inputs (no gate-margin enforcement: profiling does not
compare with the oracle), runs N sh_forward calls (default 4: three to warm up, one to capture) and
checks the device status word.  --batch overrides the workload's batch size (a reduced case of the
same kernels); --flush writes a 256 MiB buffer before every pass so that the pass starts with a
cold L2.  Argument marshalling only: every kernel is the library's own.
"""
from __future__ import annotations

import argparse

import torch

from . import binding, inputs


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("config", choices=list(inputs.CONFIGS))
    ap.add_argument("--passes", type=int, default=4)
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--flush", action="store_true")
    args = ap.parse_args()
    cfg = inputs.CONFIGS[args.config]
    inp = inputs.make_inputs(cfg, batch=args.batch, enforce_gap=False)
    layer = binding.layer_from_inputs(inp)
    x = binding.to_device(inp.x, cfg.dtype)
    out = torch.empty(inp.x.shape, dtype=torch.float32, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda") if args.flush else None
    for _ in range(args.passes):
        if flush is not None:
            flush.fill_(1)
        layer.sh_forward(x, out)
    torch.cuda.synchronize()
    assert layer.sh_last_status() == 0, "device status word set"
    print(f"{args.config}: {args.passes} passes of {inp.x.shape[0]} x {inp.x.shape[1]} tokens, {layer.sh_launch_count()} launches per pass")
    layer.close()


if __name__ == "__main__":
    main()
