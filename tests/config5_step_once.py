"""Runs the full-size config-5 step (GPT-2-small shapes, 8 x 1024 tokens) a few times through the C-ABI calls,
unchecked: the command a launch list of the step is taken from (see profiles/).  With --graph the step is
recorded once into a CUDA graph and the replays are timed.

    python tests/config5_step_once.py [--steps N] [--graph]
"""
import argparse
import os
import sys

import torch

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

import scalify_inputs as si                      # noqa: E402
from checked_ops import Ops                      # noqa: E402
from gpt_model import GPTConfig, ScaledGPT       # noqa: E402


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--steps", type=int, default=2)
    ap.add_argument("--graph", action="store_true")
    args = ap.parse_args()
    cfg = GPTConfig()
    ops = Ops(check=False)
    model = ScaledGPT(cfg, ops, seed=6)
    n = cfg.batch * cfg.seq
    ids = torch.from_numpy(si.uniform_int(6, 901, (n,), cfg.vocab)).cuda()
    tgt = torch.from_numpy(si.uniform_int(6, 902, (n,), cfg.vocab)).cuda()
    for t in (1, 2):
        model.step(ids, tgt, t=t)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if args.graph:
        stream = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            with torch.cuda.graph(graph, stream=stream):
                model.step(ids, tgt, t=3)
        graph.replay()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(args.steps):
            graph.replay()
        e1.record()
    else:
        calls = ops.calls
        e0.record()
        for t in range(3, 3 + args.steps):
            model.step(ids, tgt, t=t)
        e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    print(f"{'graph replay' if args.graph else 'eager'}: {ms:.2f} ms per step, {n / ms * 1e3:.0f} tokens/s"
          + ("" if args.graph else f", {(ops.calls - calls) // args.steps} library calls per step"))


if __name__ == "__main__":
    main()
