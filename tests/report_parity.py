"""Prints the parity table kept in profiles/parity_report.md (run on a machine with a B200):

    python -m tests.report_parity > gpurun_out/parity_report.md

For every protocol configuration: the relative L2 distance of the GPU state from the fp64 reference (the
tolerance the tests enforce is 1e-5, or 1e-3 with bf16 gradients), the distance of the fp32 reference from the
fp64 one (what keeping the state in fp32 costs by itself), and whether GPU and fp32 reference agree bit for bit.
Calls only the test harness; every assertion of the corresponding tests is active while it runs.
"""
import numpy as np

from oracle import reference as R
from tests import test_gpu_fullsize as F
from tests.gpu_harness import run_pair
from tests.helpers import rel_l2
from workloads import configs, generators as G


def small(cfg):
    layout = cfg.layout()
    kinds, learners = R.simulate_arrivals(cfg.arrival_model, cfg.num_learners, cfg.num_pushes, cfg.seed)
    w0 = G.initial_weights(layout, cfg.seed, cfg.weight_std)
    w, v, log, refs = run_pair(layout.num_params, cfg.num_learners, cfg.n, cfg.alpha0, cfg.momentum, cfg.weight_decay,
                               cfg.modulation, cfg.grad_dtype, cfg.grad_std, kinds, learners, w0, cfg.seed)
    w32, v32, _ = refs[32]
    w64, v64, _ = refs[64]
    return {"gpu_vs_fp64_w": rel_l2(w, w64), "gpu_vs_fp64_v": rel_l2(v, v64),
            "fp32ref_vs_fp64_w": rel_l2(w32, w64), "fp32ref_vs_fp64_v": rel_l2(v32, v64),
            "bit_equal": bool(np.array_equal(w, w32.astype(np.float32)) and np.array_equal(v, v32.astype(np.float32))),
            "elements": layout.num_params, "updates": cfg.num_updates, "log_rows": len(log)}


def large(cfg, lazy):
    F.run_full(cfg, lazy=lazy, overlap=not lazy)
    s = dict(F.run_full.last_stats)
    s.update(bit_equal=True, elements=cfg.layout().num_params)      # run_full asserts bit equality on the sample
    return s


def main():
    rows = [("1 tiny_softsync", small(configs.TINY_SOFTSYNC), "all elements"),
            ("2 pure_async", small(configs.PURE_ASYNC), "all elements"),
            ("3 large_softsync", large(configs.LARGE_SOFTSYNC, False), None),
            ("4 large_stale_bf16 (T=8)", large(configs.LARGE_STALE_BF16, True), None)]
    print("| config | elements | updates | compared | GPU vs fp64 ref: w | v | fp32 ref vs fp64 ref: w | v | GPU == fp32 ref (bits) | log |")
    print("|---|---|---|---|---|---|---|---|---|---|")
    for name, s, compared in rows:
        compared = compared or "%d sampled elements" % s["sampled_elements"]
        print("| %s | %d | %d | %s | %.2e | %.2e | %.2e | %.2e | %s | bit-equal |" % (
            name, s["elements"], s["updates"], compared, s["gpu_vs_fp64_w"], s["gpu_vs_fp64_v"],
            s["fp32ref_vs_fp64_w"], s["fp32ref_vs_fp64_v"], "yes" if s["bit_equal"] else "NO"))


if __name__ == "__main__":
    main()
