"""Phase trace of one decode step: where the time of the persistent forward kernel goes.

    python -m paper_2404_08856_b200.trace_phases --shape draft115m --rows 2
    python -m paper_2404_08856_b200.trace_phases --shape llava7b --layers 4 --rows 6

Builds a context whose TARGET has the requested shape (seeded random weights), prefills a short
prompt, runs a few verify steps with gamma = rows - 1 and prints, for one layer in the middle of
the model, the time CTA 0 spent in every phase (spd_trace: activation tile, weight stream,
epilogue, grid barrier for each of the four projections, attention).  The 115M draft shape with 2
rows is the kernel and the row count of a draft step.  Needs a B200 and the built library.
"""
from __future__ import annotations

import argparse
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import synth  # noqa: E402
import paper_2404_08856_b200 as spd  # noqa: E402

NAMES = ["QKV: activation tile", "QKV: weight stream", "QKV: epilogue", "barrier",
         "attention", "barrier",
         "O: activation tile", "O: weight stream", "O: epilogue", "barrier",
         "gate/up: activation tile", "gate/up: weight stream", "gate/up: epilogue", "barrier",
         "down: activation tile", "down: weight stream", "down: epilogue", "barrier"]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--shape", default="draft115m", choices=["draft115m", "llava7b", "table1"])
    ap.add_argument("--layers", type=int, default=None, help="truncate the model to this many layers")
    ap.add_argument("--rows", type=int, default=2, help="rows per step (gamma + 1), 2..8")
    ap.add_argument("--prompt", type=int, default=64)
    args = ap.parse_args()
    base = {"draft115m": synth.DRAFT_115M, "llava7b": synth.LLAVA7B_TARGET, "table1": synth.DRAFT_TABLE1}[args.shape]
    t = base if args.layers is None else synth.ModelCfg(args.layers, base.d_model, base.n_heads, base.d_ffn, base.vocab,
                                                        base.tied_embeddings, dtype="bf16")
    d = synth.ModelCfg(1, 128, 2, 344, t.vocab, True, dtype="bf16")        # a token draft: only its ids are used
    wl = synth.Workload("trace", t, d, 0, args.prompt, args.rows - 1, 16)
    tw, dw = synth.Weights(t, 1, "trace.target"), synth.Weights(d, 1, "trace.draft")
    gamma = args.rows - 1
    ctx = spd.Spd(t, d, tw.stored, dw.stored, args.prompt + 16 * args.rows + 32, 7, 1.0, True)
    ctx.prefill(None, synth.prompt_ids(wl))
    ctx.trace()                                                             # switches tracing on
    for _ in range(6):
        ctx.draft(gamma)
        ctx.verify(gamma)
    tr = ctx.trace()
    ts = (tr >> np.uint64(8)).astype(np.int64)
    ts -= ts[0]
    L = t.n_layers
    per_layer = np.zeros(18)
    for l in range(L):
        base_i = 1 + l * 18
        per_layer += np.diff(ts[base_i - 1: base_i + 18]) / 1e3
    per_layer /= L
    print(f"shape {args.shape}, {L} layers, {args.rows} rows per step: kernel {ts[-1] / 1e3:.1f} us (CTA 0's clock)")
    print("mean over layers, us:")
    for name, v in zip(NAMES, per_layer):
        print(f"  {name:28s} {v:6.2f}")
    print(f"  {'layer total':28s} {per_layer.sum():6.2f}")
    tail = ts[1 + L * 18 - 1:]
    print("after the last layer (LM head tile, stream, epilogue, barrier, statistics, barrier, rule), us:",
          " ".join(f"{x / 1e3:.2f}" for x in np.diff(tail)))
    ctx.close()


if __name__ == "__main__":
    main()
