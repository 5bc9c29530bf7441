"""Error-measurement sweep on the GPU: relative Frobenius error of each realization against the fp64
product, paired over identical operands and seeds, normalised by the cubic fp8 error (the paper's
emulated protocol, App. E.2), for the benchmark configurations.

    python -m paper_2609_26077_b200.sweep --config c1 [--scale-mode fp32|ue8m0] [--block-k 32|128]
                                          [--out sweep.jsonl] [--trials N]
    python -m paper_2609_26077_b200.sweep --summarise sweep.jsonl
    python -m paper_2609_26077_b200.sweep --ladder sweep_c7.jsonl

One JSON line is appended per (config, family, seed, realization, levels); on restart the keys that are
already in the output file are skipped.  Everything is computed by the CUDA library (fmm_matmul,
fmm_ref_gemm_fp64, fmm_error_stats); numpy only generates the seeded operands.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
from collections import defaultdict

import numpy as np

from . import fmm, realizations as P, workloads as Wl

ALL = ["cubic", "strassen", "winograd", "phi_optimal"]


def predicted(name, levels):
    """sqrt(Phi/8)^levels: the model's RMS-constant ratio against the cubic product (Sec. 2.2, Sec. 3)."""
    if name == "cubic":
        return 1.0
    return math.sqrt(P.phi(*P.get64(name)) / 8.0) ** max(levels, 1)


# name -> (M, K, N), families, trials, realizations, levels
CONFIGS = {
    "c1": dict(shape=(256, 256, 256), families=["gaussian"], trials=20, names=["cubic", "strassen"], levels=[1]),
    "c2": dict(shape=(4096, 4096, 4096), families=["gaussian", "uniform"], trials=50, names=ALL, levels=[1]),
    "c3": dict(shape=(8192, 8192, 8192), families=["gaussian"], trials=3, names=["cubic", "strassen", "phi_optimal"], levels=[1, 2]),
    "c4": dict(shape=(16384, 8192, 8192), families=["llm"], trials=3, names=ALL, levels=[1]),
    # operand-family controls (Sec. 4.3 / Table E.8): unit-variance families and Rademacher +-1 / +-10 cells
    "c6": dict(shape=(2048, 2048, 2048), families=["gaussian", "unit_uniform", "unit_laplace", "unit_t5", "rademacher", "rademacher10"],
               trials=8, names=ALL, levels=[1]),
    # the reconstructible arms of the paper's fixed panel (Table E.2): optimum, twelve Phi = 24 perturbations,
    # Strassen, Winograd form, all in the rebalanced gauge, on synthetic operands
    "c7": dict(shape=(2048, 2048, 2048), families=["gaussian", "uniform", "llm"], trials=16,
               names=["cubic"] + P.LADDER, levels=[1]),
    # orbit-ratio stability (Table E.8): fifteen exact orbit members, one shape, signed-uniform operands
    "c8": dict(shape=(2048, 2048, 2048), families=["uniform"], trials=8, names=["cubic"] + P.ORBIT15, levels=[1]),
    # weight-scale granularity (App. E.5): run with --block-k 128 and then again with --b-tile 128 [--b-bf16];
    # heterogeneous synthetic weights stand in for the stored checkpoint tiles
    "c9": dict(shape=(4096, 4096, 4096), families=["llm", "llm_hetero"], trials=8, names=ALL, levels=[1]),
    "c5": dict(shape=(2048, 2048, 2048), families=["scaled_gaussian", "student_t3"], trials=256, names=ALL, levels=[1, 2, 3]),
}


def _key(rec):
    return (rec["config"], rec["family"], rec["seed"], rec["realization"], rec["levels"], rec["scale_mode"], rec["block_k"],
            rec.get("b_tile", 0), rec.get("b_bf16", 0))


def run(args):
    import torch
    cfg = CONFIGS[args.config]
    M, K, N = cfg["shape"]
    trials = args.trials or cfg["trials"]
    done = set()
    if os.path.exists(args.out):
        for line in open(args.out):
            try:
                done.add(_key(json.loads(line)))
            except Exception:
                pass
    plans = {}

    def plan_for(name, lv):
        k = (name, lv)
        if k not in plans:
            if name == "cubic":
                plans[k] = fmm.Plan(levels=0, block_k=args.block_k, scale_mode=args.scale_mode,
                                    b_tile_n=args.b_tile, b_preround_bf16=args.b_bf16)
            else:
                plans[k] = fmm.Plan(*P.get(name), levels=lv, block_k=args.block_k, scale_mode=args.scale_mode,
                                    b_tile_n=args.b_tile, b_preround_bf16=args.b_bf16)
        return plans[k]

    out = open(args.out, "a")
    C = torch.empty((M, N), dtype=torch.float32, device="cuda")
    ref = torch.empty((M, N), dtype=torch.float64, device="cuda")
    for family in cfg["families"]:
        for seed in range(trials):
            todo = [(n, lv) for n in cfg["names"] for lv in (cfg["levels"] if n != "cubic" else [0])
                    if (args.config, family, seed, n, lv, args.scale_mode, args.block_k, args.b_tile, int(args.b_bf16)) not in done]
            if not todo:
                continue
            A, B = Wl.FAMILIES[family](M, K, N, seed)
            a, b = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
            fmm.fmm_ref_gemm_fp64(a, b, out=ref)
            for name, lv in todo:
                pl = plan_for(name, lv)
                pl.matmul(a, b, out=C)
                s = fmm.fmm_error_stats(C, ref).cpu().numpy()
                st, code = pl.device_status()
                rec = {"config": args.config, "family": family, "seed": seed, "realization": name, "levels": lv,
                       "scale_mode": args.scale_mode, "block_k": args.block_k, "b_tile": args.b_tile,
                       "b_bf16": int(args.b_bf16), "M": M, "K": K, "N": N,
                       "sum_sq_diff": float(s[0]), "sum_sq_ref": float(s[1]), "max_abs_diff": float(s[2]),
                       "rel_frobenius": float(math.sqrt(s[0] / s[1])), "device_status": code}
                out.write(json.dumps(rec) + "\n")
                out.flush()
            del a, b
    out.close()


def summarise(path, file=sys.stdout):
    """Mean per-trial error, pooled RMS error and paired ratios vs cubic, per (config, family, levels)."""
    recs = [json.loads(line) for line in open(path) if line.strip()]
    groups = defaultdict(lambda: defaultdict(dict))
    for r in recs:
        scales = r["scale_mode"] + ("+tile128" if r.get("b_tile") else "") + ("+bf16" if r.get("b_bf16") else "")
        g = (r["config"], r["family"], scales, r["block_k"])
        groups[g][(r["realization"], r["levels"])][r["seed"]] = r
    rows = []
    for g, by in sorted(groups.items()):
        cubic = by.get(("cubic", 0), {})
        for (name, lv), seeds in sorted(by.items()):
            e = np.array([seeds[s]["rel_frobenius"] for s in sorted(seeds)])
            pooled = math.sqrt(sum(seeds[s]["sum_sq_diff"] for s in seeds) / sum(seeds[s]["sum_sq_ref"] for s in seeds))
            common = [s for s in seeds if s in cubic]
            cub = np.mean([cubic[s]["rel_frobenius"] for s in common]) if common else 0.0
            # operands the cubic product represents (almost) exactly make the ratio meaningless
            ratio = np.mean([seeds[s]["rel_frobenius"] for s in common]) / cub if cub > 1e-6 else float("nan")
            pred = predicted(name, lv)
            rows.append((g, name, lv, len(e), e.mean(), e.std(), pooled, ratio, pred))
    print("| config | family | scales | blk | realization | levels | trials | mean rel. error | sd | pooled RMS | ratio vs cubic | sqrt(Phi/8)^l |", file=file)
    print("|---|---|---|---|---|---|---|---|---|---|---|---|", file=file)
    for g, name, lv, n, mean, sd, pooled, ratio, pred in rows:
        print(f"| {g[0]} | {g[1]} | {g[2]} | {g[3]} | {name} | {lv} | {n} | {mean:.5f} | {sd:.5f} | {pooled:.5f} | {ratio:.4f} | {pred:.4f} |", file=file)
    return rows


def ladder_summary(path, file=sys.stdout):
    """Panel statistics of a c7 run, per (family, scale mode, block): Spearman correlation between Phi and the
    mean error over the arms, the fraction of trials on which the optimum beats all twelve perturbations at
    once, and the relative gap between the optimum and the best arm (the paper's O2 / panel-gap statistics,
    here on synthetic operands)."""
    recs = [json.loads(line) for line in open(path) if line.strip()]
    groups = defaultdict(lambda: defaultdict(dict))
    for r in recs:
        if r["realization"] != "cubic":
            groups[(r["family"], r["scale_mode"], r["block_k"])][r["realization"]][r["seed"]] = r["rel_frobenius"]
    rows = []
    for g, by in sorted(groups.items()):
        arms = [a for a in P.LADDER if a in by]
        seeds = sorted(set.intersection(*[set(by[a]) for a in arms]))
        mean = np.array([np.mean([by[a][s] for s in seeds]) for a in arms])
        phis = np.array([P.phi(*P.get64(a)) for a in arms])
        rk = lambda x: np.argsort(np.argsort(x, kind="stable"), kind="stable").astype(float)
        # ties in Phi (the twelve arms at 24) get their average rank
        rphi = np.array([np.mean(rk(phis)[phis == v]) for v in phis])
        rho = float(np.corrcoef(rphi, rk(mean))[0, 1])
        perts = [a for a in arms if a.startswith("pert_")]
        wins = np.mean([all(by["phi_optimal_rb"][s] < by[a][s] for a in perts) for s in seeds])
        gap = float(mean[arms.index("phi_optimal_rb")] / mean.min() - 1.0)
        rows.append((g, len(seeds), rho, float(wins), gap, arms[int(mean.argmin())]))
    print("| family | scales | blk | trials | Spearman(Phi, mean error) | optimum beats all 12 perturbations | panel gap | best arm |", file=file)
    print("|---|---|---|---|---|---|---|---|", file=file)
    for g, n, rho, wins, gap, best in rows:
        print(f"| {g[0]} | {g[1]} | {g[2]} | {n} | {rho:.3f} | {wins:.3f} | {gap:.4f} | {best} |", file=file)
    return rows


def orbit_stability(path, file=sys.stdout):
    """Coefficient of variation, over the orbit members of a c8 run, of (measured error ratio against cubic) /
    sqrt(Phi/8): how stable the model's one free constant is along the orbit (Table E.8 reports 0.37 %)."""
    rows = [r for r in summarise(path, file=open(os.devnull, "w")) if r[1].startswith("orbit_")]
    out = []
    for g in sorted(set(r[0] for r in rows)):
        q = np.array([r[7] / r[8] for r in rows if r[0] == g])
        phis = np.array([r[8] ** 2 * 8 for r in rows if r[0] == g])
        out.append((g, len(q), float(phis.min()), float(phis.max()), float(q.mean()), float(q.std(ddof=1) / q.mean())))
    print("| family | scales | blk | members | Phi range | mean measured/predicted | CV |", file=file)
    print("|---|---|---|---|---|---|---|", file=file)
    for g, n, lo, hi, m, cv in out:
        print(f"| {g[1]} | {g[2]} | {g[3]} | {n} | {lo:.2f} - {hi:.2f} | {m:.4f} | {100 * cv:.2f} % |", file=file)
    return out


def covariance_diagnostic(names=("strassen", "winograd", "phi_optimal", "strassen_rb", "winograd_rb", "phi_optimal_rb"),
                          n=512, seeds=4, block_k=128, scale_mode="fp32", family="gaussian", file=sys.stdout):
    """Cross-term covariance diagnostic (App. D.1): the part of the error that is linear in the rounding
    residuals is L_q = sum_r W[r][q] t_r with t_r = dx_r y_r + x_r dy_r (x_r, y_r the encoded combinations,
    dx_r, dy_r their quantization residuals).  The model keeps only the diagonal sum_{r,q} W[r][q]^2 |t_r|_F^2
    (that is what defines Phi); the fraction (|L|_F^2 - diag) / |L|_F^2 measures what the dropped cross terms
    contribute.  The quantized operands come from the CUDA encoder; the algebra around them is fp64 numpy.
    The paper reports armwise means between -0.085 % and 0.201 % (n = 512, Gaussian, four seeds, 1 x 128 groups)."""
    import torch
    rows = []
    for name in names:
        U, V, W = (np.asarray(x, dtype=np.float64) for x in P.get(name))
        plan = fmm.Plan(*P.get(name), levels=1, block_k=block_k, scale_mode=scale_mode)
        fr = []
        for seed in range(seeds):
            A, B = Wl.FAMILIES[family](n, n, n, seed)
            ws = plan.workspace(n, n, n)
            plan.encode_only(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), workspace=ws)
            torch.cuda.synchronize()
            h = n // 2
            Aq = [A[:h, :h], A[:h, h:], A[h:, :h], A[h:, h:]]
            Bq = [B[:h, :h], B[:h, h:], B[h:, :h], B[h:, h:]]
            t = []
            for r in range(U.shape[0]):
                x = sum(U[r, j] * Aq[j].astype(np.float64) for j in range(4))
                y = sum(V[r, j] * Bq[j].astype(np.float64) for j in range(4))
                ca, sa = plan.quantized_operand(ws, n, n, n, r, "A")
                cb, sb = plan.quantized_operand(ws, n, n, n, r, "B")
                if scale_mode != "fp32":
                    sa, sb = np.ldexp(1.0, sa.astype(np.int32) - 127), np.ldexp(1.0, sb.astype(np.int32) - 127)
                dec = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()
                xh = dec[ca] * np.repeat(sa.astype(np.float64), block_k, axis=1)
                yh = dec[cb] * np.repeat(sb.astype(np.float64), block_k, axis=0)
                t.append((xh - x) @ y + x @ (yh - y))
            Lsq = sum(np.linalg.norm(sum(W[r, q] * t[r] for r in range(len(t)))) ** 2 for q in range(4))
            diag = sum(W[r, q] ** 2 * np.linalg.norm(t[r]) ** 2 for r in range(len(t)) for q in range(4))
            fr.append((Lsq - diag) / Lsq)
        plan.close()
        rows.append((name, float(np.mean(fr)), float(np.min(fr)), float(np.max(fr))))
    print(f"| realization | mean residual fraction | min | max |  (n = {n}, {family}, {seeds} seeds, {scale_mode} blk {block_k})", file=file)
    print("|---|---|---|---|", file=file)
    for name, m, lo, hi in rows:
        print(f"| {name} | {100 * m:+.3f} % | {100 * lo:+.3f} % | {100 * hi:+.3f} % |", file=file)
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", choices=sorted(CONFIGS))
    ap.add_argument("--scale-mode", default="fp32", choices=["fp32", "ue8m0"])
    ap.add_argument("--block-k", type=int, default=32, choices=[32, 128])
    ap.add_argument("--b-tile", type=int, default=0, choices=[0, 128], help="weight-side 128 x 128 scale tiles (blk 128, fp32)")
    ap.add_argument("--b-bf16", action="store_true", help="bf16 pre-round of each encoded weight combination")
    ap.add_argument("--out", default="sweep.jsonl")
    ap.add_argument("--trials", type=int, default=0)
    ap.add_argument("--summarise")
    ap.add_argument("--ladder", help="panel statistics of a c7 output file")
    ap.add_argument("--orbit", help="orbit-ratio stability of a c8 output file")
    ap.add_argument("--covariance", action="store_true", help="cross-term covariance diagnostic (n = 512, four seeds)")
    a = ap.parse_args()
    if a.summarise:
        summarise(a.summarise)
    elif a.ladder:
        ladder_summary(a.ladder)
    elif a.orbit:
        orbit_stability(a.orbit)
    elif a.covariance:
        covariance_diagnostic(block_k=a.block_k, scale_mode=a.scale_mode)
    else:
        if not a.config:
            ap.error("--config or --summarise is required")
        run(a)


if __name__ == "__main__":
    main()
