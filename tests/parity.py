"""Helpers of the GPU-vs-oracle parity tests: shared set-up and the comparison rules.

Rules (tolerances stated here once):
  * idx / qjl bits: bit-exact, except coordinates whose oracle value (fp64) lies within
    WINDOW = 1e-5 (in units of ||x||) of a decision boundary; the mismatch rate over the
    remaining coordinates must be <= MAX_MISMATCH = 1e-4.
  * qjl and gamma are compared conditioned on the GPU's idx (one flipped idx inside the window
    legitimately changes the residual): the oracle recomputes r, gamma, sign(S r) from that idx.
  * gamma, norms, reconstructions, scores: relative 1e-4 (fp32 arithmetic against fp64); for
    scores the scale is max(|est|, ||q|| nu) because an estimate can be near 0.
"""
from __future__ import annotations

import math

import numpy as np
import torch

import paper_2504_19874_b200 as tq
from oracle import turboquant_oracle as orc

WINDOW = 1e-5
MAX_MISMATCH = 1e-4
RTOL = 1e-4


class Setup:
    """Oracle-made global parameters (Pi, S, fp32 codebook) and the matching GPU plan."""

    def __init__(self, d, bits, mode, pi_seed=42, s_seed=43, layout=None, centroids=None):
        self.d, self.bits, self.mode = d, bits, mode
        self.layout = layout
        self.mse_bits = bits - 1 if mode == tq.TQ_PROD else bits
        self.Pi = orc.rotation(d, pi_seed).astype(np.float32)
        self.S = orc.projection(d, s_seed).astype(np.float32) if mode == tq.TQ_PROD else None
        self.c = (orc.codebook(d, self.mse_bits) if centroids is None else np.asarray(centroids)).astype(np.float32)
        self.t = (0.5 * (self.c[:-1].astype(np.float64) + self.c[1:].astype(np.float64)))
        self.plan = tq.Plan(d, bits, mode, self.Pi, self.S, self.c)
        if layout is not None:
            self.plan.set_layout(layout)
        self.idx_rb = tq.tq_idx_row_bytes(d, self.mse_bits)
        self.qjl_rb = tq.tq_qjl_row_bytes(d)

    # ---- GPU calls ---------------------------------------------------------------------
    def quantize(self, X: torch.Tensor, with_norms=True, scratch_bytes=None):
        n = X.shape[0]
        dev = X.device
        idx = torch.full((n, max(self.idx_rb, 1)), 0xAB, dtype=torch.uint8, device=dev)
        norms = torch.full((n,), -7.0, dtype=torch.float32, device=dev) if with_norms else None
        ws = scratch_bytes if scratch_bytes is not None else tq.tq_workspace_bytes(self.plan, tq.TQ_OP_QUANTIZE, n)
        scratch = torch.empty(max(ws, 16), dtype=torch.uint8, device=dev)
        if self.mode == tq.TQ_MSE:
            tq.tq_quantize_mse(self.plan, X, idx, norms, scratch)
            qjl = gamma = None
        else:
            qjl = torch.full((n, self.qjl_rb), 0xCD, dtype=torch.uint8, device=dev)
            gamma = torch.full((n,), -7.0, dtype=torch.float32, device=dev)
            tq.tq_quantize_prod(self.plan, X, idx, qjl, gamma, norms, scratch)
        tq.tq_plan_status(self.plan)
        return idx, qjl, gamma, norms

    def dequantize(self, n, idx, qjl, gamma, norms):
        Xh = torch.empty((n, self.d), dtype=torch.float32, device=idx.device)
        tq.tq_dequantize(self.plan, n, idx, qjl, gamma, norms, Xh)
        torch.cuda.synchronize()
        return Xh

    def score(self, Q, n, idx, qjl, gamma, norms):
        nq = Q.shape[0]
        scores = torch.empty((nq, n), dtype=torch.float32, device=Q.device)
        ws = torch.empty(max(tq.tq_workspace_bytes(self.plan, tq.TQ_OP_SCORE, n, nq), 16), dtype=torch.uint8, device=Q.device)
        tq.tq_score(self.plan, Q, n, idx, qjl, gamma, norms, scores, ws)
        torch.cuda.synchronize()
        return scores

    def topk(self, Q, n, idx, qjl, gamma, norms, k, workspace_bytes=None):
        nq = Q.shape[0]
        ts = torch.empty((nq, k), dtype=torch.float32, device=Q.device)
        ti = torch.empty((nq, k), dtype=torch.int32, device=Q.device)
        wb = workspace_bytes or tq.tq_workspace_bytes(self.plan, tq.TQ_OP_TOPK, n, nq, k)
        ws = torch.empty(max(wb, 16), dtype=torch.uint8, device=Q.device)
        tq.tq_topk(self.plan, Q, n, idx, qjl, gamma, norms, k, ts, ti, ws)
        torch.cuda.synchronize()
        return ts, ti


def as_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float64).numpy()


def nibble_rows_to_coordinates(idx: np.ndarray, qjl: np.ndarray, d: int):
    """The nibble layout read literally from its definition: nibble j of the row [idx row | qjl row] holds
    coordinate j, index in its low three bits and the sign bit on top.  Returns (index [n, d], bit [n, d]) and
    the nibbles beyond d (which must be zero)."""
    row = np.concatenate([idx, qjl], axis=1)
    nib = np.stack([row & 15, row >> 4], axis=2).reshape(row.shape[0], -1)
    return nib[:, :d] & 7, nib[:, :d] >> 3, nib[:, d:]


def unpack(su: Setup, idx, qjl):
    if getattr(su, "layout", None) == tq.TQ_LAYOUT_NIBBLE:
        i3, bit, _ = nibble_rows_to_coordinates(idx.cpu().numpy(), qjl.cpu().numpy(), su.d)
        return i3.astype(np.uint8), bit.astype(np.int8) * 2 - 1
    idx_np = orc.unpack_bits(idx.cpu().numpy(), su.mse_bits, su.d) if su.mse_bits > 0 else \
        np.zeros((idx.shape[0], su.d), dtype=np.uint8)
    z_np = None
    if qjl is not None:
        z_np = orc.unpack_bits(qjl.cpu().numpy(), 1, su.d).astype(np.int8) * 2 - 1
    return idx_np, z_np


def check_pad_bits_zero(packed: torch.Tensor, bits: int, d: int):
    p = packed.cpu().numpy()
    used = d * bits
    assert not p[:, (used + 7) // 8:].any(), "pad bytes must be zero"
    if used % 8:
        assert not (p[:, used // 8] >> (used % 8)).any(), "pad bits must be zero"


def check_quantize(su: Setup, X: torch.Tensor, idx, qjl, gamma, norms, unit_input=False):
    """Codes, gamma and norms of the GPU against the oracle.  Returns a dict of rates."""
    Xd = as_f64(X)
    n = Xd.shape[0]
    idx_gpu, z_gpu = unpack(su, idx, qjl)
    nibble = getattr(su, "layout", None) == tq.TQ_LAYOUT_NIBBLE
    if nibble:
        assert not nibble_rows_to_coordinates(idx.cpu().numpy(), qjl.cpu().numpy(), su.d)[2].any(), "pad nibbles must be zero"
    elif su.mse_bits > 0:
        check_pad_bits_zero(idx, su.mse_bits, su.d)
    nu_orc = np.sqrt(np.sum(Xd * Xd, axis=1))
    if norms is not None:
        nu_gpu = as_f64(norms)
        assert np.all(np.abs(nu_gpu - nu_orc) <= RTOL * nu_orc), "norms differ"
    if unit_input:          # the library quantises the rows as they are
        U, scale = Xd, np.ones(n)
    else:
        scale = np.where(nu_orc > 0, nu_orc, 1.0)
        U = Xd / scale[:, None]
    Y = orc.rotate(U, su.Pi)
    idx_orc = orc.nearest_centroid(Y, su.c) if su.mse_bits > 0 else np.zeros_like(idx_gpu)
    if su.mse_bits > 0:
        margin = np.min(np.abs(Y[:, :, None] - su.t[None, None, :]), axis=2)
    else:
        margin = np.full(Y.shape, np.inf)
    inside = margin <= WINDOW
    diff = idx_gpu != idx_orc
    stats = {"idx_excluded": inside.mean(), "idx_mismatch": (diff & ~inside).sum() / max((~inside).sum(), 1),
             "idx_flips_in_window": int((diff & inside).sum())}
    assert stats["idx_mismatch"] <= MAX_MISMATCH, stats
    # a flip inside the window must still land on an adjacent cell
    assert np.all(np.abs(idx_gpu.astype(int) - idx_orc.astype(int))[diff] == 1)
    if su.mode == tq.TQ_PROD:
        if not nibble:
            check_pad_bits_zero(qjl, 1, su.d)
        ok_rows = ~np.any(diff & ~inside, axis=1)
        # unit_input: feed the oracle rows that it will not rescale
        Xo = U if unit_input else Xd
        z_orc, gamma_orc, P = orc.qjl_given_idx(Xo, idx_gpu, su.Pi, su.S, su.c)
        near = np.abs(P) <= WINDOW
        zdiff = (z_gpu != z_orc) & ok_rows[:, None]
        denom = max(((~near) & ok_rows[:, None]).sum(), 1)
        stats["qjl_excluded"] = near.mean()
        stats["qjl_mismatch"] = (zdiff & ~near).sum() / denom
        assert stats["qjl_mismatch"] <= MAX_MISMATCH, stats
        g_gpu = as_f64(gamma)
        assert np.all(np.abs(g_gpu - gamma_orc)[ok_rows] <= RTOL * np.maximum(gamma_orc[ok_rows], 1e-30) + 1e-12), "gamma differs"
        # unconditioned rate (against the oracle's own idx), reported only
        z_full, _, _ = orc.qjl_given_idx(Xo, idx_orc, su.Pi, su.S, su.c)
        stats["qjl_mismatch_unconditioned"] = (z_gpu != z_full).mean()
    return stats


def oracle_dequant(su: Setup, idx, qjl, gamma, norms):
    idx_np, z_np = unpack(su, idx, qjl)
    n = idx_np.shape[0]
    nu = as_f64(norms) if norms is not None else np.ones(n)
    if su.mode == tq.TQ_MSE:
        return orc.dequant_mse(idx_np, nu, su.Pi, su.c)
    return orc.dequant_prod(idx_np, z_np, as_f64(gamma), nu, su.Pi, su.S, su.c)


def check_dequant(su: Setup, Xhat_gpu, idx, qjl, gamma, norms):
    ref = oracle_dequant(su, idx, qjl, gamma, norms)
    got = as_f64(Xhat_gpu)
    err = np.linalg.norm(got - ref, axis=1)
    nrm = np.linalg.norm(ref, axis=1)
    assert np.all(err <= RTOL * nrm + 1e-30), float(np.max(err / np.maximum(nrm, 1e-30)))
    return ref


def score_tolerance(su: Setup, Q, norms, n):
    # |sum_j q'_j c[idx_j]| <= ||q|| ||c[idx]|| ~ ||q||, so ||q|| nu is the scale of an estimate
    nu = as_f64(norms) if norms is not None else np.ones(n)
    qn = np.linalg.norm(as_f64(Q), axis=1)
    return RTOL * qn[:, None] * nu[None, :]


def check_scores(su: Setup, scores_gpu, Q, idx, qjl, gamma, norms):
    """Estimates against <q, DeQuant(code)> taken in the original basis by the oracle."""
    Xh = oracle_dequant(su, idx, qjl, gamma, norms)
    ref = orc.score(as_f64(Q), Xh)
    got = as_f64(scores_gpu)
    tol = np.maximum(RTOL * np.abs(ref), score_tolerance(su, Q, norms, Xh.shape[0]))
    assert np.all(np.abs(got - ref) <= tol), float(np.max(np.abs(got - ref) / tol))
    return ref


def check_topk(ref_scores, tol, top_s, top_i, k):
    """ids must match the oracle's as a set once near-ties around the k-th value are set aside;
    every returned score must be the oracle's score of the returned id; order must be descending."""
    top_s, top_i = as_f64(top_s), top_i.cpu().numpy().astype(np.int64)
    ref_vals, ref_ids = orc.topk(ref_scores, k)
    for q in range(ref_scores.shape[0]):
        ids = top_i[q]
        assert len(set(ids.tolist())) == k and ids.min() >= 0 and ids.max() < ref_scores.shape[1]
        t = tol[q].max() if np.ndim(tol) == 2 else tol
        assert np.all(np.abs(top_s[q] - ref_scores[q, ids]) <= np.maximum(t, RTOL * np.abs(top_s[q])))
        assert np.all(np.diff(top_s[q]) <= 0)
        kth = ref_vals[q, -1]
        must = set(np.nonzero(ref_scores[q] > kth + 2 * t)[0].tolist())
        may = set(np.nonzero(ref_scores[q] >= kth - 2 * t)[0].tolist())
        got = set(ids.tolist())
        assert must <= got <= may, (q, len(must - got), len(got - may))
