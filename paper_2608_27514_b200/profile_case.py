"""Runs one stage of the verification step a few times on a small, seeded case: the target of the
ncu captures summarised under profiles/ (small enough for a full-set capture, larger than L2).

  python -m paper_2608_27514_b200.profile_case topk [--rows 2048] [--vocab 126464] [--k 3]
  python -m paper_2608_27514_b200.profile_case attention [--workload cfg4] [--batch 4]

Prints the CUDA-event time of the last call.  Nothing here is timed for the benchmark.
"""
import argparse

import torch

from . import binding as B
from . import workloads as W
from .step import VerifyStep


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("stage", choices=["topk", "attention"])
    ap.add_argument("--rows", type=int, default=2048)
    ap.add_argument("--vocab", type=int, default=126464)
    ap.add_argument("--k", type=int, default=3)
    ap.add_argument("--workload", default="cfg4")
    ap.add_argument("--batch", type=int, default=4)
    ap.add_argument("--calls", type=int, default=4)
    args = ap.parse_args()
    dev = "cuda:0"
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if args.stage == "topk":
        g = torch.Generator(device=dev).manual_seed(0)
        x = (torch.randn((args.rows, args.vocab), generator=g, device=dev) * 3).bfloat16()
        conf = torch.empty(args.rows, device=dev)
        idx = torch.empty((args.rows, args.k), dtype=torch.int32, device=dev)
        prob = torch.empty((args.rows, args.k), device=dev)
        lse = torch.empty(args.rows, device=dev)
        ws = torch.empty(max(16, B.tsd_confidence_topk_workspace_bytes(args.rows, args.vocab, args.k)),
                         dtype=torch.uint8, device=dev)
        call = lambda: B.tsd_confidence_topk(x, args.k, conf, idx, prob, lse, ws)
        work, unit = args.rows * args.vocab * 2 / 1e9, "GB"
    else:
        cfg = W.small(W.CONFIGS[args.workload], S=args.batch)
        attn = W.attention_inputs(cfg, dev)
        st = VerifyStep.for_config(cfg, dev)
        st.build_mask()
        call = lambda: st.attention(attn["q"], attn["k_cache"], attn["v_cache"], attn["k_draft"],
                                    attn["v_draft"], attn["sm_scale"])
        work, unit = 4.0 * cfg.rows * (cfg.Nc + cfg.R) * cfg.d * cfg.Hq / 1e12, "TFLOP"
    for _ in range(args.calls - 1):
        call()
    torch.cuda.synchronize()
    e0.record()
    call()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    print("%s: %.4f ms, %.1f %s/s" % (args.stage, ms, work / (ms * 1e-3), unit))


if __name__ == "__main__":
    main()
