"""Distortion of the two quantisers measured through the CUDA library (Section 4.1 of the paper:
the quantities its validation plots show, here on synthetic data).

    python -m paper_2504_19874_b200.distortion [--d 1536] [--n 20000]

prints, per bit width b = 1..4, the mean squared reconstruction error of TurboQuant_mse on unit
vectors (Theorem 1: between 4^-b and sqrt(3) pi / 2 * 4^-b; about 0.36, 0.117, 0.03, 0.009) and the
bias and mean squared error of the inner-product estimate of TurboQuant_prod (Theorem 2: unbiased,
error about 1.57/d, 0.56/d, 0.18/d, 0.047/d for unit queries), plus the multiplicative bias of the
mse reconstruction used as an inner-product estimator (Section 3.2: 2/pi at b = 1).
"""
from __future__ import annotations

import argparse
import math

import torch

from . import binding as tq


def _unit_rows(n: int, d: int, seed: int, dev, decay: float = 0.5, offset: float = 0.3):
    """Anisotropic, offset, unit-normalised rows (the law of the embedding-like configurations)."""
    g = torch.Generator(device=dev).manual_seed(seed)
    X = torch.randn((n, d), generator=g, device=dev) * torch.arange(1, d + 1, device=dev, dtype=torch.float32) ** -decay
    X = X / X.norm(dim=1, keepdim=True)
    mu = torch.randn(d, generator=g, device=dev)
    X = X + offset * mu / mu.norm()
    return (X / X.norm(dim=1, keepdim=True)).contiguous()


def measure(d: int = 1536, n: int = 20000, nq: int = 8, device: str = "cuda:0", seed: int = 0, isotropic: bool = True):
    """Returns {b: {...}} for b = 1..4; every number comes from tq_quantize_*, tq_dequantize and tq_score.

    With one fixed (Pi, S) the estimator's error on a direction shared by all vectors is one fixed number, so the
    bias figures are meaningful for isotropic rows only (the default); isotropic=False uses the anisotropic, offset
    law of the embedding-like configurations, on which the distortion levels must be the same (data-oblivious)."""
    dev = torch.device(device)
    Pi = tq.tq_rotation(d, 42 + seed)
    S = tq.tq_rotation(d, 43 + seed, tq.TQ_GAUSSIAN)
    if isotropic:
        X = _unit_rows(n, d, 1 + seed, dev, decay=0.0, offset=0.0)
        Q = _unit_rows(nq, d, 1001 + seed, dev, decay=0.0, offset=0.0)
    else:
        X = _unit_rows(n, d, 1 + seed, dev)
        Q = _unit_rows(nq, d, 1001 + seed, dev)
    exact = (Q.double() @ X.double().T)                     # [nq, n]
    out = {}
    for b in (1, 2, 3, 4):
        res = {}
        # ---- TurboQuant_mse at b bits
        cent, _ = tq.tq_codebook(d, b)
        plan = tq.Plan(d, b, tq.TQ_MSE, Pi, None, cent)
        idx = torch.empty((n, plan.idx_row_bytes), dtype=torch.uint8, device=dev)
        norms = torch.empty(n, device=dev)
        scratch = torch.empty(max(tq.tq_workspace_bytes(plan, tq.TQ_OP_QUANTIZE, n), 16), dtype=torch.uint8, device=dev)
        tq.tq_quantize_mse(plan, X, idx, norms, scratch)
        Xh = torch.empty((n, d), device=dev)
        tq.tq_dequantize(plan, n, idx, None, None, norms, Xh)
        res["dmse"] = float(((X.double() - Xh.double()) ** 2).sum(1).mean())
        est = (Q.double() @ Xh.double().T)
        res["mse_estimator_slope"] = float((est * exact).sum() / (exact * exact).sum())   # multiplicative bias
        # ---- TurboQuant_prod at b bits (b - 1 bits of indices + 1 bit of QJL signs)
        cent_p, _ = tq.tq_codebook(d, b - 1)
        plan_p = tq.Plan(d, b, tq.TQ_PROD, Pi, S, cent_p)
        idx_p = torch.empty((n, max(plan_p.idx_row_bytes, 1)), dtype=torch.uint8, device=dev)
        qjl = torch.empty((n, plan_p.qjl_row_bytes), dtype=torch.uint8, device=dev)
        gamma = torch.empty(n, device=dev)
        scratch = torch.empty(max(tq.tq_workspace_bytes(plan_p, tq.TQ_OP_QUANTIZE, n), 16), dtype=torch.uint8, device=dev)
        tq.tq_quantize_prod(plan_p, X, idx_p, qjl, gamma, norms, scratch)
        scores = torch.empty((nq, n), device=dev)
        ws = torch.empty(max(tq.tq_workspace_bytes(plan_p, tq.TQ_OP_SCORE, n, nq), 16), dtype=torch.uint8, device=dev)
        tq.tq_score(plan_p, Q, n, idx_p, qjl, gamma, norms, scores, ws)
        err = scores.double() - exact
        res["dprod_times_d"] = float((err ** 2).mean()) * d
        res["prod_bias"] = float(err.mean())
        res["prod_bias_sigma"] = float(err.std()) / math.sqrt(err.numel())
        res["prod_slope"] = float((scores.double() * exact).sum() / (exact * exact).sum())
        # error against the size of the inner product: correlation of err^2 with exact^2 (Section 4.1: the variance
        # of the prod estimator does not grow with the inner product)
        e2, x2 = err ** 2, exact ** 2
        res["prod_err_vs_ip_corr"] = float(((e2 - e2.mean()) * (x2 - x2.mean())).mean() / (e2.std() * x2.std()))
        torch.cuda.synchronize()
        out[b] = res
    return out


def recall_1_at_k(d: int = 1536, n: int = 100000, nq: int = 256, bits=(2, 4), ks=(1, 2, 4, 8, 16, 32, 64),
                  device: str = "cuda:0", seed: int = 0):
    """Recall 1@k of nearest-neighbour search by inner product (the measure of the paper's nearest-neighbour
    experiments): the fraction of queries whose exact top-1 vector (fp32 scan of the original rows) is among the
    k best of tq_topk on the TurboQuant_prod codes.  Returns {b: {k: recall}}."""
    dev = torch.device(device)
    Pi = tq.tq_rotation(d, 42 + seed)
    S = tq.tq_rotation(d, 43 + seed, tq.TQ_GAUSSIAN)
    X = _unit_rows(n, d, 1 + seed, dev)
    Q = _unit_rows(nq, d, 1001 + seed, dev)
    truth = torch.argmax(Q @ X.T, dim=1)
    kmax = max(ks)
    out = {}
    for b in bits:
        cent, _ = tq.tq_codebook(d, b - 1)
        plan = tq.Plan(d, b, tq.TQ_PROD, Pi, S, cent)
        idx = torch.empty((n, max(plan.idx_row_bytes, 1)), dtype=torch.uint8, device=dev)
        qjl = torch.empty((n, plan.qjl_row_bytes), dtype=torch.uint8, device=dev)
        gamma = torch.empty(n, device=dev)
        norms = torch.empty(n, device=dev)
        scratch = torch.empty(max(tq.tq_workspace_bytes(plan, tq.TQ_OP_QUANTIZE, n), 16), dtype=torch.uint8, device=dev)
        tq.tq_quantize_prod(plan, X, idx, qjl, gamma, norms, scratch)
        ts = torch.empty((nq, kmax), device=dev)
        ti = torch.empty((nq, kmax), dtype=torch.int32, device=dev)
        ws = torch.empty(max(tq.tq_workspace_bytes(plan, tq.TQ_OP_TOPK, n, nq, kmax), 16), dtype=torch.uint8, device=dev)
        tq.tq_topk(plan, Q, n, idx, qjl, gamma, norms, kmax, ts, ti, ws)
        hit = ti.long() == truth[:, None]
        out[b] = {k: float(hit[:, :k].any(dim=1).float().mean()) for k in ks}
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--d", type=int, default=1536)
    ap.add_argument("--n", type=int, default=20000)
    ap.add_argument("--anisotropic", action="store_true", help="embedding-like rows (bias columns are then not meaningful)")
    args = ap.parse_args()
    r = measure(args.d, args.n, isotropic=not args.anisotropic)
    print(f"d = {args.d}, n = {args.n} unit vectors, 8 unit queries")
    print(" b   D_mse   [4^-b, 2.72*4^-b]     D_prod*d   bias (sigma)            slope_prod  slope_mse")
    for b, v in r.items():
        print(f" {b}  {v['dmse']:.4f}  [{4.0 ** -b:.4f}, {2.7207 * 4.0 ** -b:.4f}]   {v['dprod_times_d']:8.4f}   "
              f"{v['prod_bias']:+.2e} ({v['prod_bias_sigma']:.1e})   {v['prod_slope']:.4f}      {v['mse_estimator_slope']:.4f}")
    rec = recall_1_at_k(args.d)
    print("recall 1@k of tq_topk on TurboQuant_prod codes (100,000 embedding-like rows, 256 queries):")
    for b, v in rec.items():
        print(f" b = {b}: " + "  ".join(f"1@{k} = {x:.3f}" for k, x in v.items()))


if __name__ == "__main__":
    main()
