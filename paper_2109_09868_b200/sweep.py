"""Parameter sweep on synthetic stand-ins, mirroring the grid of the paper's experiments
(Section 4.2: K in {8,10,12}, S in {0..3}, E in {1,2,3}; Appendix B: noise sigma in {1,10,100})
without its datasets or trained networks.

    python -m paper_2109_09868_b200.sweep [--groups 4096] [--classes 10] [--json]

For every (K, S, E, sigma, model) cell the whole pipeline runs on the GPU through the library:
encode hidden queries -> seeded stand-in model (linear, or linear + softmax) on the coded queries ->
drop S stragglers, corrupt E workers with N(0, sigma^2) noise -> locate -> decode from the trusted
workers.  Reported per cell: how often the located set equals the injected set, the decode error
against the model applied to the uncoded queries, and how often the arg-max class agrees with it
(the paper's accuracy metric, Section 4.1 "Performance metric").
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import binding as ap


def run_cell(K: int, S: int, E: int, sigma: float, softmax: bool, G: int, C: int, d_in: int, seed: int, dev,
             keep_tensors: bool = False) -> dict:
    W = 2 * (K + E) + S if E > 0 else K + S
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)
    X = torch.rand((G, K, d_in), generator=gen, device=dev)
    M = torch.randn((d_in, C), generator=gen, device=dev) / np.sqrt(d_in) * 3.0

    def f(x):
        y = x @ M
        return torch.softmax(y, dim=-1) if softmax else y

    p = ap.make_params(K, W, E)
    Yt = f(ap.approxifer_encode(p, X)).contiguous()
    rng = np.random.default_rng(seed)
    order = rng.random((G, W)).argsort(axis=1)
    absent = order[:, :S]
    bad = np.sort(order[:, S:S + E], axis=1)
    mask = np.full(G, (1 << W) - 1, dtype=np.uint64)
    for s in range(S):
        mask &= ~(np.uint64(1) << absent[:, s].astype(np.uint64))
    mask = mask.astype(np.uint32)
    if E > 0:
        noise = torch.randn((G, E, C), generator=gen, device=dev) * sigma
        rows = torch.arange(G, device=dev)[:, None].expand(G, E)
        Yt[rows, torch.as_tensor(bad, device=dev)] += noise
        adv, trusted = ap.approxifer_locate(p, Yt, ap.mask_tensor(mask, dev))
        recall = float((adv.cpu().numpy() == bad).all(axis=1).mean())
    else:
        adv, trusted, recall = None, ap.mask_tensor(mask, dev), float("nan")
    Yh = ap.approxifer_decode(p, Yt, trusted)
    Y = f(X)
    err = (Yh - Y).abs().amax(dim=(1, 2)) / Y.abs().amax(dim=(1, 2))
    agree = float((Yh.argmax(-1) == Y.argmax(-1)).float().mean())
    out = {"K": K, "S": S, "E": E, "W": W, "sigma": sigma, "model": "softmax" if softmax else "linear",
           "located_equals_injected": recall, "decode_rel_err_median": float(err.median()),
           "decode_rel_err_max": float(err.max()), "argmax_agreement": agree}
    if keep_tensors:  # (for the tests: what went into and came out of the library)
        out["tensors"] = {"Yt": Yt, "mask": mask, "injected": bad, "adv": adv, "trusted": trusted, "Yhat": Yh}
    if 2 <= K + E <= 13 and 2 * (K + E) <= W:
        # Algorithm 3 on the same corrupted predictions: P/Q at the alpha nodes, nothing located
        Yr = ap.approxifer_decode_rational(p, Yt, ap.mask_tensor(mask, dev))
        err_r = (Yr - Y).abs().amax(dim=(1, 2)) / Y.abs().amax(dim=(1, 2))
        err_r = torch.nan_to_num(err_r, nan=float("inf"))
        out["rational_rel_err_median"] = float(err_r.median())
        out["rational_argmax_agreement"] = float((Yr.argmax(-1) == Y.argmax(-1)).float().mean())
    return out


def main():
    pa = argparse.ArgumentParser()
    pa.add_argument("--groups", type=int, default=4096)
    pa.add_argument("--classes", type=int, default=10)
    pa.add_argument("--d-in", type=int, default=64)
    pa.add_argument("--json", action="store_true")
    args = pa.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("the sweep runs the CUDA library: a GPU is required")
    dev = torch.device("cuda:0")
    cells = []
    for softmax in (False, True):
        for K in (8, 10, 12):
            for S in (0, 1, 2, 3):
                cells.append(run_cell(K, S, 0, 0.0, softmax, args.groups, args.classes, args.d_in, 1000 + K * 10 + S, dev))
            for E in (1, 2, 3):
                for sigma in (1.0, 10.0, 100.0):
                    if 2 * (K + E) <= 32:
                        cells.append(run_cell(K, 0, E, sigma, softmax, args.groups, args.classes, args.d_in,
                                              2000 + K * 100 + E * 10 + int(sigma), dev))
    if args.json:
        print(json.dumps(cells))
        return
    print("| model | K | S | E | W | sigma | located == injected | decode rel. err (median / max) | arg-max agreement "
          "| Algorithm 3: rel. err (median) / arg-max agreement |")
    print("|---|---|---|---|---|---|---|---|---|---|")
    for c in cells:
        rat = "-" if "rational_rel_err_median" not in c else "%.3g / %.3f" % (c["rational_rel_err_median"],
                                                                              c["rational_argmax_agreement"])
        print("| %s | %d | %d | %d | %d | %g | %s | %.3g / %.3g | %.3f | %s |" % (
            c["model"], c["K"], c["S"], c["E"], c["W"], c["sigma"],
            "-" if c["E"] == 0 else "%.4f" % c["located_equals_injected"],
            c["decode_rel_err_median"], c["decode_rel_err_max"], c["argmax_agreement"], rat))


if __name__ == "__main__":
    main()
