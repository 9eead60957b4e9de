"""KV-cache decode over a compressed cache (third evaluation configuration): K quantised with
TurboQuant_prod, V with TurboQuant_mse, 128 channels per head split into 64 outlier channels at 3
bits and 64 regular channels at 2 bits, 32 query heads (4 per KV head), softmax(q K^T / sqrt(128)) V.
GPU: tq_quantize_*, tq_score, tq_softmax, tq_wsum.  Oracle: dequantise the same codes, textbook
attention in fp64."""
import math

import numpy as np
import pytest
import torch

import paper_2504_19874_b200 as tq
import tq_workloads as wl
from oracle import turboquant_oracle as orc
from tests import parity as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
HEAD_DIM, GROUP = 128, 64
# Attention outputs (relative L2 error per output row) and softmax weights (relative, per weight) against the fp64
# oracle on the same codes.  Measured worst cases at the full shape of the KV configuration (8 x 32,768 tokens):
# outputs 2.1e-6 (separate calls), 2.1e-6 (fused), fused against separate 2.7e-6, weights 4.1e-6; the other
# shapes and bit widths of this file 0.5e-6 .. 2.2e-6.  The bounds are about four times that: the logits are
# fp32 sums of ~128 terms of magnitude up to ~30, i.e. ~1e-6 absolute after the 1/sqrt(128) scale, and the
# weights and outputs inherit exactly that.
S5_TOL = 1e-5
S5_TOL_WEIGHTS = 2e-5


def split_channels(Xh: torch.Tensor):
    """Outlier / regular channel lists of one head (harness rule: largest energy over tokens)."""
    out = orc.select_outlier_channels(Xh.double().cpu().numpy(), GROUP)
    rest = np.setdiff1d(np.arange(HEAD_DIM), out)
    return torch.from_numpy(out).to(DEV), torch.from_numpy(rest).to(DEV)


def attend_gpu(groupsK, groupsV, Kh, Vh, Qh):
    """One KV head: returns out [4, 128] fp32 and everything the oracle needs to redo it."""
    T = Kh.shape[0]
    scores, rec = [], {"K": [], "V": []}
    chK, chV = split_channels(Kh), split_channels(Vh)
    for su, ch in zip(groupsK, chK):
        Xg = Kh[:, ch].contiguous()
        codes = su.quantize(Xg)
        rec["K"].append((su, ch, Xg, codes))
        scores.append(su.score(Qh[:, ch].contiguous(), T, *codes))
    W = torch.empty_like(scores[0])
    tq.tq_softmax(scores[0], scores[1], 1.0 / math.sqrt(HEAD_DIM), W)
    out = torch.zeros((Qh.shape[0], HEAD_DIM), device=DEV)
    for su, ch in zip(groupsV, chV):
        Xg = Vh[:, ch].contiguous()
        codes = su.quantize(Xg)
        rec["V"].append((su, ch, Xg, codes))
        og = torch.empty((Qh.shape[0], GROUP), device=DEV)
        ws = torch.empty(tq.tq_workspace_bytes(su.plan, tq.TQ_OP_WSUM, T, Qh.shape[0]), dtype=torch.uint8, device=DEV)
        tq.tq_wsum(su.plan, W, T, *codes, og, ws)
        out[:, ch] = og
    torch.cuda.synchronize()
    return out, W, rec


def attend_oracle(rec, Qh):
    T = rec["K"][0][2].shape[0]
    Khat, Vhat = np.zeros((T, HEAD_DIM)), np.zeros((T, HEAD_DIM))
    for su, ch, _, codes in rec["K"]:
        Khat[:, ch.cpu().numpy()] = P.oracle_dequant(su, *codes)
    for su, ch, _, codes in rec["V"]:
        Vhat[:, ch.cpu().numpy()] = P.oracle_dequant(su, *codes)
    s = orc.score(P.as_f64(Qh), Khat)
    return orc.attend(s, Vhat, 1.0 / math.sqrt(HEAD_DIM)), s


@pytest.fixture(scope="module")
def groups():
    gK = (P.Setup(GROUP, 3, tq.TQ_PROD, 72, 73), P.Setup(GROUP, 2, tq.TQ_PROD, 74, 75))
    gV = (P.Setup(GROUP, 3, tq.TQ_MSE, 76, 77), P.Setup(GROUP, 2, tq.TQ_MSE, 78, 79))
    return gK, gV


def test_kv_decode_full_shape(groups):
    gK, gV = groups
    K, V, Q = wl.kv_cache(device=DEV)                      # [8, 32768, 128] x2, [32, 128], bf16
    heads, T, _ = K.shape
    worst = 0.0
    for h in range(heads):
        Qh = Q[4 * h:4 * h + 4]
        out, W, rec = attend_gpu(gK, gV, K[h], V[h], Qh)
        ref, s = attend_oracle(rec, Qh)
        # softmax weights against the oracle's, then the output rows
        p = np.exp(s / math.sqrt(HEAD_DIM) - (s / math.sqrt(HEAD_DIM)).max(axis=1, keepdims=True))
        p /= p.sum(axis=1, keepdims=True)
        wdev = np.abs(P.as_f64(W) - p) / np.maximum(p, 1e-9)
        worst_w = max(locals().get("worst_w", 0.0), float(wdev[p > 1e-9].max()))
        assert np.allclose(P.as_f64(W), p, rtol=S5_TOL_WEIGHTS, atol=1e-9)
        err = np.linalg.norm(P.as_f64(out) - ref, axis=1) / np.linalg.norm(ref, axis=1)
        worst = max(worst, float(err.max()))
        if h == 0:   # codes of the four groups of one head against the oracle's quantiser
            for kind in ("K", "V"):
                for su, _, Xg, codes in rec[kind]:
                    st = P.check_quantize(su, Xg, *codes)
                    assert st["idx_mismatch"] == 0
    # logits carry the fp32 score error (<= 1e-4 of ||q|| nu) times 1/sqrt(128); weights and outputs inherit it
    print(f"S5 measured: separate calls, full shape: output {worst:.3e}, weights {worst_w:.3e}")
    assert worst <= S5_TOL, worst


def test_wsum_matches_dequantised_sum_all_modes():
    g = torch.Generator(device="cpu").manual_seed(11)
    for d, bits, mode, n, nw in [(64, 3, tq.TQ_PROD, 1000, 4), (64, 2, tq.TQ_MSE, 129, 1), (200, 4, tq.TQ_PROD, 515, 11),
                                 (24, 1, tq.TQ_PROD, 70, 3), (128, 4, tq.TQ_MSE, 300, 9)]:
        su = P.Setup(d, bits, mode)
        X = (torch.randn((n, d), generator=g) * 2).to(DEV)
        codes = su.quantize(X)
        W = torch.randn((nw, n), generator=g).to(DEV)
        out = torch.empty((nw, d), device=DEV)
        ws = torch.empty(tq.tq_workspace_bytes(su.plan, tq.TQ_OP_WSUM, n, nw), dtype=torch.uint8, device=DEV)
        tq.tq_wsum(su.plan, W, n, *codes, out, ws)
        out2 = torch.empty_like(out)
        tq.tq_wsum(su.plan, W, n, *codes, out2, ws)
        torch.cuda.synchronize()
        assert torch.equal(out, out2)
        ref = P.as_f64(W) @ P.oracle_dequant(su, *codes)
        scale = np.abs(P.as_f64(W)) @ np.linalg.norm(P.oracle_dequant(su, *codes), axis=1)
        assert np.all(np.linalg.norm(P.as_f64(out) - ref, axis=1) <= P.RTOL * scale)


def test_softmax_rows_and_empty_inputs():
    g = torch.Generator(device="cpu").manual_seed(12)
    s1 = (torch.randn((5, 3001), generator=g) * 20).to(DEV)
    s2 = (torch.randn((5, 3001), generator=g) * 20).to(DEV)
    W = torch.empty_like(s1)
    tq.tq_softmax(s1, s2, 0.37, W)
    ref = torch.softmax((s1.double() + s2.double()) * 0.37, dim=1)
    assert torch.allclose(W.double(), ref, rtol=1e-4, atol=1e-12)
    tq.tq_softmax(s1, None, 1.0, W)
    assert torch.allclose(W.double(), torch.softmax(s1.double(), dim=1), rtol=1e-4, atol=1e-12)
    su = P.Setup(64, 2, tq.TQ_MSE)
    out = torch.full((2, 64), 7.0, device=DEV)
    tq.tq_wsum(su.plan, None, 0, None, None, None, None, out, None)     # n = 0: zeros
    torch.cuda.synchronize()
    assert not bool(out.any())


# ---------------------------------------------------------------------------------------------
# tq_attend_decode: the same computation for all KV heads and channel groups of a layer in one call


def _fused_layer(groupsK, groupsV, recs, Q, heads, T, qpk):
    """Concatenates the per-head codes of `recs` head-major and runs tq_attend_decode."""
    groups = []
    for gi in range(len(groupsK)):
        cat = lambda kind, i: (None if recs[0][kind][gi][3][i] is None
                               else torch.cat([recs[h][kind][gi][3][i] for h in range(heads)]).contiguous())
        groups.append({
            "plan_k": groupsK[gi].plan, "plan_v": groupsV[gi].plan,
            "k_idx": cat("K", 0), "k_qjl": cat("K", 1), "k_gamma": cat("K", 2), "k_norms": cat("K", 3),
            "v_idx": cat("V", 0), "v_norms": cat("V", 3),
            "k_channels": torch.stack([recs[h]["K"][gi][1] for h in range(heads)]).to(torch.int32).contiguous(),
            "v_channels": torch.stack([recs[h]["V"][gi][1] for h in range(heads)]).to(torch.int32).contiguous(),
        })
    d = groupsK[0].d
    ws = torch.empty(tq.tq_attend_decode_workspace_bytes(len(groups), heads, T, d), dtype=torch.uint8, device=DEV)
    out = torch.full((heads * qpk, HEAD_DIM), float("nan"), device=DEV)
    tq.tq_attend_decode(groups, heads, T, qpk, Q, 1.0 / math.sqrt(HEAD_DIM), out, ws)
    out2 = torch.full_like(out, float("nan"))
    tq.tq_attend_decode(groups, heads, T, qpk, Q, 1.0 / math.sqrt(HEAD_DIM), out2, ws)
    torch.cuda.synchronize()
    assert torch.equal(out, out2)          # fixed reduction orders: repeatable bit for bit
    return out


def test_fused_decode_full_shape_against_the_separate_calls(groups):
    gK, gV = groups
    K, V, Q = wl.kv_cache(device=DEV)
    heads, T, _ = K.shape
    outs, recs = [], []
    for h in range(heads):
        out, _, rec = attend_gpu(gK, gV, K[h], V[h], Q[4 * h:4 * h + 4])
        outs.append(out)
        recs.append(rec)
    ref = torch.cat(outs)
    fused = _fused_layer(gK, gV, recs, Q, heads, T, 4)
    err = (fused - ref).norm(dim=1) / ref.norm(dim=1)
    print(f"S5 measured: fused vs separate calls, full shape: {float(err.max()):.3e}")
    assert float(err.max()) <= S5_TOL, float(err.max())
    orc_ref = np.concatenate([attend_oracle(recs[h], Q[4 * h:4 * h + 4])[0] for h in range(heads)])
    err_o = np.linalg.norm(P.as_f64(fused) - orc_ref, axis=1) / np.linalg.norm(orc_ref, axis=1)
    print(f"S5 measured: fused vs oracle, full shape: {float(err_o.max()):.3e}")
    assert float(err_o.max()) <= S5_TOL, float(err_o.max())


# (1, 140000, 2): 547 slices of 256 tokens, more than the merge kernel's 512 threads take in one round
@pytest.mark.parametrize("heads,T,qpk", [(2, 2500, 3), (1, 1024, 1), (3, 77, 4), (1, 140000, 2)])
def test_fused_decode_against_the_oracle(groups, heads, T, qpk):
    gK, gV = groups
    K, V, Q = wl.kv_cache(heads=heads, tokens=T, q_per_kv=qpk, seed=5 + T, device=DEV)
    recs, refs = [], []
    for h in range(heads):
        Qh = Q[qpk * h:qpk * h + qpk]
        _, _, rec = attend_gpu(gK, gV, K[h], V[h], Qh)
        recs.append(rec)
        refs.append(attend_oracle(rec, Qh)[0])
    ref = np.concatenate(refs)
    fused = P.as_f64(_fused_layer(gK, gV, recs, Q, heads, T, qpk))
    err = np.linalg.norm(fused - ref, axis=1) / np.linalg.norm(ref, axis=1)
    print(f"S5 measured: fused vs oracle heads={heads} T={T}: {float(err.max()):.3e}")
    assert float(err.max()) <= S5_TOL, float(err.max())


@pytest.mark.parametrize("d,specs,unit_norm", [
    (32, [(4, tq.TQ_PROD, 4), (3, tq.TQ_MSE, 1), (1, tq.TQ_PROD, 2), (2, tq.TQ_PROD, 3)], False),   # four groups of 32 channels
    (96, [(3, tq.TQ_PROD, 3)], False),                                                                # one group of 96
    (64, [(4, tq.TQ_PROD, 4), (3, tq.TQ_PROD, 3)], False),                                            # the 3.5-bit split
    (64, [(3, tq.TQ_PROD, 3), (2, tq.TQ_PROD, 2)], True),                                             # rows of unit norm, no norm arrays
])
def test_fused_decode_group_shapes(d, specs, unit_norm):
    """Group counts, group widths, bit widths and quantiser kinds other than the configuration's, fp32 queries,
    a head stride larger than the token count and a ragged last slice.  specs: (key bits, key quantiser, value bits)."""
    ng, heads, T, qpk, cap = len(specs), 3, 777, 3, 801
    hd = ng * d
    gK = [P.Setup(d, kb, km, 90 + 2 * i, 91 + 2 * i) for i, (kb, km, vb) in enumerate(specs)]
    gV = [P.Setup(d, vb, tq.TQ_MSE, 70 + 2 * i, 71 + 2 * i) for i, (kb, km, vb) in enumerate(specs)]
    g = torch.Generator(device="cpu").manual_seed(1000 + d + ng)
    K = torch.randn((heads, T, hd), generator=g).to(DEV)
    V = torch.randn((heads, T, hd), generator=g).to(DEV)
    Q = torch.randn((heads * qpk, hd), generator=g).to(DEV)
    perm = [torch.randperm(hd, generator=g).to(DEV) for _ in range(heads)]      # arbitrary channel lists
    gds, Khat, Vhat = [], np.zeros((heads, T, hd)), np.zeros((heads, T, hd))
    for gi in range(ng):
        suk, suv = gK[gi], gV[gi]
        gd = {"plan_k": suk.plan, "plan_v": suv.plan,
              "k_idx": torch.zeros((heads * cap, max(suk.idx_rb, 1)), dtype=torch.uint8, device=DEV),
              "k_qjl": torch.zeros((heads * cap, suk.qjl_rb), dtype=torch.uint8, device=DEV) if suk.mode == tq.TQ_PROD else None,
              "k_gamma": torch.zeros(heads * cap, device=DEV) if suk.mode == tq.TQ_PROD else None,
              "k_norms": None if unit_norm else torch.zeros(heads * cap, device=DEV),
              "v_idx": torch.zeros((heads * cap, suv.idx_rb), dtype=torch.uint8, device=DEV),
              "v_norms": None if unit_norm else torch.zeros(heads * cap, device=DEV),
              "k_channels": torch.stack([perm[h][gi * d:(gi + 1) * d] for h in range(heads)]).to(torch.int32).contiguous(),
              "v_channels": torch.stack([perm[h][gi * d:(gi + 1) * d] for h in range(heads)]).to(torch.int32).contiguous()}
        if suk.mse_bits == 0:
            gd["k_idx"] = None
        for h in range(heads):
            ch = perm[h][gi * d:(gi + 1) * d]
            Xk, Xv = K[h][:, ch].contiguous(), V[h][:, ch].contiguous()
            if unit_norm:
                Xk, Xv = Xk / Xk.norm(dim=1, keepdim=True), Xv / Xv.norm(dim=1, keepdim=True)
            ck, cv = suk.quantize(Xk, with_norms=not unit_norm), suv.quantize(Xv, with_norms=not unit_norm)
            r = slice(h * cap, h * cap + T)
            if gd["k_idx"] is not None:
                gd["k_idx"][r] = ck[0]
            if suk.mode == tq.TQ_PROD:
                gd["k_qjl"][r], gd["k_gamma"][r] = ck[1], ck[2]
            gd["v_idx"][r] = cv[0]
            if not unit_norm:
                gd["k_norms"][r], gd["v_norms"][r] = ck[3], cv[3]
            Khat[h][:, ch.cpu().numpy()] = P.oracle_dequant(suk, *ck)
            Vhat[h][:, ch.cpu().numpy()] = P.oracle_dequant(suv, *cv)
        gds.append(gd)
    ws = torch.empty(tq.tq_attend_decode_workspace_bytes(ng, heads, T, d), dtype=torch.uint8, device=DEV)
    out = torch.full((heads * qpk, hd), float("nan"), device=DEV)
    scale = 1.0 / math.sqrt(hd)
    tq.tq_attend_decode(gds, heads, T, qpk, Q, scale, out, ws, head_stride=cap)
    torch.cuda.synchronize()
    ref = np.concatenate([orc.attend(orc.score(P.as_f64(Q[qpk * h:qpk * h + qpk]), Khat[h]), Vhat[h], scale) for h in range(heads)])
    err = np.linalg.norm(P.as_f64(out) - ref, axis=1) / np.linalg.norm(ref, axis=1)
    print(f"S5 measured: fused vs oracle d={d} groups={specs} unit_norm={unit_norm}: {float(err.max()):.3e}")
    assert float(err.max()) <= S5_TOL, float(err.max())


def test_fused_decode_with_codebooks_that_are_not_antisymmetric():
    """The tensor-core kernels expand an antisymmetric codebook over the index bits; any other codebook (the API
    accepts what the caller passes) takes the table-lookup kernel.  Same check against the oracle."""
    def skewed(bits):
        c = orc.codebook(GROUP, bits).copy()
        c[0] *= 1.05
        c[-1] *= 0.97
        return c
    gK = (P.Setup(GROUP, 3, tq.TQ_PROD, 72, 73, centroids=skewed(2)), P.Setup(GROUP, 2, tq.TQ_PROD, 74, 75, centroids=skewed(1)))
    gV = (P.Setup(GROUP, 3, tq.TQ_MSE, 76, 77, centroids=skewed(3)), P.Setup(GROUP, 2, tq.TQ_MSE, 78, 79, centroids=skewed(2)))
    heads, T, qpk = 2, 1300, 4
    K, V, Q = wl.kv_cache(heads=heads, tokens=T, q_per_kv=qpk, seed=17, device=DEV)
    recs, refs = [], []
    for h in range(heads):
        Qh = Q[qpk * h:qpk * h + qpk]
        _, _, rec = attend_gpu(gK, gV, K[h], V[h], Qh)
        recs.append(rec)
        refs.append(attend_oracle(rec, Qh)[0])
    ref = np.concatenate(refs)
    fused = P.as_f64(_fused_layer(gK, gV, recs, Q, heads, T, qpk))
    err = np.linalg.norm(fused - ref, axis=1) / np.linalg.norm(ref, axis=1)
    print(f"S5 measured: fused (table-lookup kernel) vs oracle: {float(err.max()):.3e}")
    assert float(err.max()) <= S5_TOL, float(err.max())


def test_fused_decode_other_bit_widths_and_argument_checks():
    # one group of 128 channels: keys TurboQuant_mse 4-bit (no QJL part), values 4-bit; then keys prod 4-bit (3-bit indices)
    for kbits, kmode, vbits in ((4, tq.TQ_MSE, 4), (4, tq.TQ_PROD, 1), (1, tq.TQ_PROD, 2), (2, tq.TQ_MSE, 3)):
        gK = (P.Setup(HEAD_DIM, kbits, kmode, 81, 82),)
        gV = (P.Setup(HEAD_DIM, vbits, tq.TQ_MSE, 83, 84),)
        heads, T, qpk = 2, 1500, 2
        K, V, Q = wl.kv_cache(heads=heads, tokens=T, q_per_kv=qpk, seed=9, device=DEV)
        ch = torch.arange(HEAD_DIM, device=DEV)
        recs, refs = [], []
        for h in range(heads):
            rec = {"K": [], "V": []}
            Kh, Vh = K[h].float().contiguous(), V[h].float().contiguous()
            rec["K"].append((gK[0], ch, Kh, gK[0].quantize(Kh)))
            rec["V"].append((gV[0], ch, Vh, gV[0].quantize(Vh)))
            recs.append(rec)
            refs.append(attend_oracle(rec, Q[qpk * h:qpk * h + qpk])[0])
        fused = P.as_f64(_fused_layer(gK, gV, recs, Q, heads, T, qpk))
        ref = np.concatenate(refs)
        err = np.linalg.norm(fused - ref, axis=1) / np.linalg.norm(ref, axis=1)
        print(f"S5 measured: fused vs oracle kbits={kbits} mode={kmode} vbits={vbits}: {float(err.max()):.3e}")
        assert float(err.max()) <= S5_TOL, (kbits, kmode, vbits, float(err.max()))
    with pytest.raises(tq.TqError):     # a workspace that is too small is refused
        g = {"plan_k": gK[0].plan, "plan_v": gV[0].plan, "k_idx": recs[0]["K"][0][3][0], "k_qjl": recs[0]["K"][0][3][1],
             "k_gamma": recs[0]["K"][0][3][2], "k_norms": recs[0]["K"][0][3][3], "v_idx": recs[0]["V"][0][3][0],
             "v_norms": recs[0]["V"][0][3][3], "k_channels": ch.to(torch.int32).repeat(1, 1), "v_channels": ch.to(torch.int32).repeat(1, 1)}
        tq.tq_attend_decode([g], 1, T, qpk, Q, 1.0, torch.empty((qpk, HEAD_DIM), device=DEV),
                            torch.empty(256, dtype=torch.uint8, device=DEV))


def test_streaming_append_then_decode(groups):
    """A cache of capacity 300 tokens per head: 200 tokens quantised in one batch, 10 more appended one at a
    time with tq_kv_append; the appended rows against the oracle's quantiser and the batch quantiser, then
    decode attention over the 210 tokens against the oracle."""
    gK, gV = groups
    heads, T0, T1, cap, qpk = 2, 200, 210, 300, 4
    K, V, Q = wl.kv_cache(heads=heads, tokens=T1, q_per_kv=qpk, seed=21, device=DEV)
    chK = [split_channels(K[h][:T0]) for h in range(heads)]
    chV = [split_channels(V[h][:T0]) for h in range(heads)]
    gds = []
    for gi in range(2):
        suk, suv = gK[gi], gV[gi]
        gd = {"plan_k": suk.plan, "plan_v": suv.plan,
              "k_idx": torch.zeros((heads * cap, suk.idx_rb), dtype=torch.uint8, device=DEV),
              "k_qjl": torch.zeros((heads * cap, suk.qjl_rb), dtype=torch.uint8, device=DEV),
              "k_gamma": torch.zeros(heads * cap, device=DEV), "k_norms": torch.zeros(heads * cap, device=DEV),
              "v_idx": torch.zeros((heads * cap, suv.idx_rb), dtype=torch.uint8, device=DEV),
              "v_norms": torch.zeros(heads * cap, device=DEV),
              "k_channels": torch.stack([chK[h][gi] for h in range(heads)]).to(torch.int32).contiguous(),
              "v_channels": torch.stack([chV[h][gi] for h in range(heads)]).to(torch.int32).contiguous()}
        for h in range(heads):
            ck = suk.quantize(K[h][:T0][:, chK[h][gi]].contiguous())
            cv = suv.quantize(V[h][:T0][:, chV[h][gi]].contiguous())
            r = slice(h * cap, h * cap + T0)
            gd["k_idx"][r], gd["k_qjl"][r], gd["k_gamma"][r], gd["k_norms"][r] = ck
            gd["v_idx"][r], gd["v_norms"][r] = cv[0], cv[3]
        gds.append(gd)
    for t in range(T0, T1):
        tq.tq_kv_append(gds, heads, cap, t, K[:, t].contiguous(), V[:, t].contiguous())
    torch.cuda.synchronize()
    # the appended rows: against the oracle's quantiser (same criteria as the batch path) and the batch quantiser
    recs = []
    for h in range(heads):
        rec = {"K": [], "V": []}
        for gi in range(2):
            suk, suv = gK[gi], gV[gi]
            new = slice(h * cap + T0, h * cap + T1)
            Xk = K[h][T0:T1][:, chK[h][gi]].contiguous()
            Xv = V[h][T0:T1][:, chV[h][gi]].contiguous()
            app_k = (gds[gi]["k_idx"][new].contiguous(), gds[gi]["k_qjl"][new].contiguous(),
                     gds[gi]["k_gamma"][new].contiguous(), gds[gi]["k_norms"][new].contiguous())
            app_v = (gds[gi]["v_idx"][new].contiguous(), None, None, gds[gi]["v_norms"][new].contiguous())
            P.check_quantize(suk, Xk, *app_k)
            P.check_quantize(suv, Xv, *app_v)
            bk, bv = suk.quantize(Xk), suv.quantize(Xv)
            assert (bk[0] != app_k[0]).float().mean() <= 0.01 and (bv[0] != app_v[0]).float().mean() <= 0.01
            assert torch.allclose(bk[3], app_k[3], rtol=1e-6) and torch.allclose(bk[2], app_k[2], rtol=1e-4)
            allr = slice(h * cap, h * cap + T1)
            rec["K"].append((suk, chK[h][gi], K[h][:T1][:, chK[h][gi]], tuple(gds[gi][k][allr].contiguous() for k in ("k_idx", "k_qjl", "k_gamma", "k_norms"))))
            rec["V"].append((suv, chV[h][gi], V[h][:T1][:, chV[h][gi]], (gds[gi]["v_idx"][allr].contiguous(), None, None, gds[gi]["v_norms"][allr].contiguous())))
        recs.append(rec)
    ws = torch.empty(tq.tq_attend_decode_workspace_bytes(2, heads, T1, GROUP), dtype=torch.uint8, device=DEV)
    out = torch.zeros((heads * qpk, HEAD_DIM), device=DEV)
    tq.tq_attend_decode(gds, heads, T1, qpk, Q, 1.0 / math.sqrt(HEAD_DIM), out, ws, head_stride=cap)
    torch.cuda.synchronize()
    ref = np.concatenate([attend_oracle(recs[h], Q[qpk * h:qpk * h + qpk])[0] for h in range(heads)])
    err = np.linalg.norm(P.as_f64(out) - ref, axis=1) / np.linalg.norm(ref, axis=1)
    print(f"S5 measured: appended cache, fused vs oracle: {float(err.max()):.3e}")
    assert float(err.max()) <= S5_TOL, float(err.max())
    with pytest.raises(tq.TqError):
        tq.tq_kv_append(gds, heads, cap, cap, K[:, 0].contiguous(), V[:, 0].contiguous())   # position outside the cache


def test_fused_decode_edge_cases(groups):
    """No tokens (zero rows), fp32 queries with a row stride, an output with a row stride, and repeatability
    across different head strides."""
    gK, gV = groups
    heads, T, qpk = 2, 300, 2
    K, V, Q = wl.kv_cache(heads=heads, tokens=T, q_per_kv=qpk, seed=31, device=DEV)
    recs = []
    for h in range(heads):
        _, _, rec = attend_gpu(gK, gV, K[h], V[h], Q[qpk * h:qpk * h + qpk])
        recs.append(rec)
    base = _fused_layer(gK, gV, recs, Q, heads, T, qpk)
    # the same codes in a cache of larger capacity, fp32 queries inside a wider buffer, output inside a wider buffer
    cap = 512
    gds = []
    for gi in range(2):
        gd = {"plan_k": gK[gi].plan, "plan_v": gV[gi].plan}
        for name, kind, i in (("k_idx", "K", 0), ("k_qjl", "K", 1), ("k_gamma", "K", 2), ("k_norms", "K", 3), ("v_idx", "V", 0), ("v_norms", "V", 3)):
            src = [recs[h][kind][gi][3][i] for h in range(heads)]
            buf = torch.zeros((heads * cap,) + tuple(src[0].shape[1:]), dtype=src[0].dtype, device=DEV)
            for h in range(heads):
                buf[h * cap:h * cap + T] = src[h]
            gd[name] = buf
        gd["k_channels"] = torch.stack([recs[h]["K"][gi][1] for h in range(heads)]).to(torch.int32).contiguous()
        gd["v_channels"] = torch.stack([recs[h]["V"][gi][1] for h in range(heads)]).to(torch.int32).contiguous()
        gds.append(gd)
    Qw = torch.zeros((heads * qpk, HEAD_DIM + 24), device=DEV)
    Qw[:, :HEAD_DIM] = Q.float()
    outw = torch.full((heads * qpk, HEAD_DIM + 8), 5.0, device=DEV)
    ws = torch.empty(tq.tq_attend_decode_workspace_bytes(2, heads, T, GROUP), dtype=torch.uint8, device=DEV)
    tq.tq_attend_decode(gds, heads, T, qpk, Qw[:, :HEAD_DIM], 1.0 / math.sqrt(HEAD_DIM), outw[:, :HEAD_DIM], ws, head_stride=cap)
    torch.cuda.synchronize()
    assert torch.equal(outw[:, :HEAD_DIM], base)          # bf16 queries are exact in fp32: identical results
    assert bool((outw[:, HEAD_DIM:] == 5.0).all())        # nothing written outside the named columns
    out0 = torch.full((heads * qpk, HEAD_DIM), 3.0, device=DEV)
    tq.tq_attend_decode(gds, heads, 0, qpk, Q, 1.0, out0, ws, head_stride=cap)
    torch.cuda.synchronize()
    assert not bool(out0.any())
    tq.tq_attend_decode(gds, 0, T, qpk, Q, 1.0, out0, ws, head_stride=cap)   # no heads: nothing to do
