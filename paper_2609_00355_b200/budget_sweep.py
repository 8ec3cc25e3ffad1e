"""Budget sweep on synthetic match probabilities: accepted length and round time against the verify budget N,
chain against tree (the shape of the paper's budget tables: width saturates, the verify pass is flat in N).

    python -m paper_2609_00355_b200.budget_sweep [--config 7b] [--steps 48] [--p-m 0.8 0.5]

Candidates are calibrated: the true next token sits at rank r of its depth with the probability the controlled
marginal gives that rank, so sibling branches can be hit.  Every (k, N) point builds its own engine on the same
weights, prefills the same context, replays one CUDA graph per round and prints one JSON line.
"""
import argparse
import json
import statistics

import torch

from . import build as glance_build
from . import synth
from .round_driver import RoundBench


def run_point(cfg, weights, dev, steps, warmup=3):
    b = RoundBench(cfg, dev, weights=weights)
    b.calibrated = True
    eng = b.eng
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ms, committed = [], 0
    for step in range(warmup + steps):
        Y = b.lookahead()
        b.make_candidates(Y)
        b.cand_ids.copy_(b.ids_host)
        if step == 1:
            torch.cuda.synchronize()
            b.capture_round()
        torch.cuda.synchronize()
        start.record()
        b.round_device()
        stop.record()
        torch.cuda.synchronize()
        if step >= warmup:
            ms.append(start.elapsed_time(stop))
            committed += int(eng.accept_len.sum().item()) + cfg.batch
    eng.check_device_status()
    return {"k": cfg.topk, "N": cfg.tree_N, "p_m": cfg.p_m, "tau": committed / steps,
            "ms_per_round": sum(ms) / steps, "ms_median": statistics.median(ms),
            "tokens_per_s": committed / (sum(ms) * 1e-3)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="7b")
    ap.add_argument("--steps", type=int, default=48)
    ap.add_argument("--p-m", type=float, nargs="+", default=[0.8, 0.5])
    args = ap.parse_args()
    assert torch.cuda.is_available(), "the budget sweep needs a CUDA device (there is no CPU fallback)"
    glance_build.build()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    base = synth.CONFIGS[args.config]
    torch.manual_seed(0)
    weights = synth.make_weights(base, dev)
    for p_m in args.p_m:
        for k, N in [(1, 16), (base.topk, 16), (base.topk, 32), (base.topk, 48), (base.topk, 64)]:
            cfg = base.replace(tree_N=N, topk=k, p_m=p_m, name=f"{base.name}-k{k}-N{N}")
            print(json.dumps(run_point(cfg, weights, dev, args.steps)), flush=True)


if __name__ == "__main__":
    main()
