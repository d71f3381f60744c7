"""Run a few forward calls of one synthetic workload, for use under a profiler.

    python -m paper_1712_01084_b200.run_case cfg5 --k 128 --batch 1 --calls 6
    python -m paper_1712_01084_b200.run_case cfg2 --calls 6
    python -m paper_1712_01084_b200.run_case cfg3 --batch 8 --calls 4 [--one-kernel]
    python -m paper_1712_01084_b200.run_case cfg4 --steps 64 --calls 2
    python -m paper_1712_01084_b200.run_case cfg5 --k 32 --batch 20 --no-tile      # chunked matrix-vector kernel
    python -m paper_1712_01084_b200.run_case cfg5 --k 128 --batch 128 --tile-kernel 2     # clustered tile kernel

Calls rotate over `--copies` independent copies of the layer(s) (default: enough to exceed twice the L2, at
most 4) so that a profiled launch does not find its weights in L2.  Plain launches on the current stream, one
synchronise at the end; prints the kernel the library picked.  Only the library is exercised: nothing is checked
here (the tests do that).
"""
from __future__ import annotations

import argparse

import numpy as np


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("case", choices=["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"])
    ap.add_argument("--k", type=int, default=128, help="cfg5: kept tiles per block-row (of 128)")
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256, help="cfg4: recurrent steps per call")
    ap.add_argument("--calls", type=int, default=6)
    ap.add_argument("--copies", type=int, default=0)
    ap.add_argument("--one-kernel", action="store_true", help="cfg3: the whole chain as one cooperative kernel")
    ap.add_argument("--no-tile", action="store_true", help="keep fp16 B=64 layers off the tensor-core tile path")
    ap.add_argument("--no-pdl", action="store_true", help="launch without programmatic stream serialization")
    ap.add_argument("--tile-kernel", type=int, default=1, choices=[0, 1, 2, 3],
                    help="tensor-core tile kernel (tuning key 12): 1 automatic, 0 one block-row per CTA, 2 clustered, 3 persistent")
    args = ap.parse_args()

    import torch
    from . import binding as pb
    from . import synth

    pb.lib()
    if args.no_tile:
        pb.pp_set_tuning(9, 0)
    if args.no_pdl:
        pb.pp_set_tuning(8, 0)
    if args.one_kernel:
        pb.pp_set_tuning(14, 1)
    pb.pp_set_tuning(12, args.tile_kernel)      # before any layer exists: the persistent kernel's plan is built at creation
    l2 = 126 * 2 ** 20

    def copies_for(weight_bytes):
        return args.copies if args.copies > 0 else max(1, min(4, -(-2 * l2 // max(1, weight_bytes)) + 1))

    if args.case == "cfg3":
        wl = synth.config3(batch=args.batch)
        R = copies_for(sum(l.T * l.B * l.B * 2 for l in wl.layers))
        chains = []
        for _ in range(R):
            layers = [pb.Layer.from_synth(l) for l in wl.layers] if not chains else [l.clone() for l in chains[0].layers]
            chains.append(pb.Chain(layers, [l.act for l in wl.layers], max_batch=max(8, args.batch)))
        x = torch.from_numpy(wl.x).cuda()
        y = torch.empty((args.batch, wl.layers[-1].M), dtype=torch.float32, device="cuda")
        for i in range(args.calls):
            pb.pp_chain_forward(chains[i % R], x, out=y)
        torch.cuda.synchronize()
        print(f"cfg3 chain, batch {args.batch}, {'one kernel' if args.one_kernel else 'one launch per layer'}, "
              f"{args.calls} calls over {R} copies; status {chains[0].status()}")
        return
    if args.case == "cfg4":
        wl = synth.config4(steps=args.steps)
        lay, H, I = wl.layers[0], wl.extra["H"], wl.extra["I"]
        L = pb.Layer.from_synth(lay)
        cell = pb.Lstm(L, I, H, max_steps=args.steps)
        xs = torch.from_numpy(wl.x).cuda()
        h = torch.zeros(H, dtype=torch.float16, device="cuda")
        c = torch.zeros(H, dtype=torch.float32, device="cuda")
        for _ in range(args.calls):
            pb.pp_lstm_forward(cell, xs, h, c)
        torch.cuda.synchronize()
        print(f"cfg4 recurrent cell, {args.steps} steps per call, {args.calls} calls; status {cell.status()}")
        return
    wl = {"cfg1": lambda: synth.config1(batch=args.batch), "cfg2": lambda: synth.config2(batch=args.batch),
          "cfg5": lambda: synth.config5(k=args.k, batch=args.batch)}[args.case]()
    lay = wl.layers[0]
    first = pb.Layer.from_synth(lay)
    R = copies_for(lay.T * lay.B * lay.B * lay.tile_values.dtype.itemsize)
    layers = [first] + [first.clone() for _ in range(R - 1)]
    x = torch.from_numpy(np.ascontiguousarray(wl.x)).cuda()
    y = torch.empty((args.batch, lay.M), dtype=torch.float32, device="cuda")
    for i in range(args.calls):
        pb.pp_forward(layers[i % R], x, lay.act, out=y)
    torch.cuda.synchronize()
    print(f"{wl.name}, batch {args.batch}: {first.launch_info(args.batch)}; {args.calls} calls over {R} copies; "
          f"status {first.status()}")


if __name__ == "__main__":
    main()
