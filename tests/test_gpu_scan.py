"""The packed-code scan on the integer tensor path (d >= 128) against the oracle: every bit width of
both variants, ragged sizes, each query-count configuration, and the three top-k flows (dense
blocks, pilot threshold + filter, overflow rescue)."""
import numpy as np
import pytest
import torch

import paper_2504_19874_b200 as tq
import tq_workloads as wl
from tests import parity as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _data(d, n, nq, seed):
    g = torch.Generator(device="cpu").manual_seed(seed)
    X = (torch.randn((n, d), generator=g) * torch.rand((n, 1), generator=g).mul(2).add(0.3)).to(DEV)
    Q = (torch.randn((nq, d), generator=g) * torch.rand((nq, 1), generator=g).mul(4).add(0.1)).to(DEV)
    return X, Q


@pytest.mark.parametrize("d", [128, 200, 520, 1536])
@pytest.mark.parametrize("bits,mode", [(1, tq.TQ_MSE), (2, tq.TQ_MSE), (3, tq.TQ_MSE), (4, tq.TQ_MSE), (1, tq.TQ_PROD),
                                       (2, tq.TQ_PROD), (3, tq.TQ_PROD), (4, tq.TQ_PROD), (5, tq.TQ_PROD)])
def test_scores_every_bit_width(d, bits, mode):
    su = P.Setup(d, bits, mode)
    n = 300 if d == 1536 else 777
    X, Q = _data(d, n, 5, 1000 * d + 10 * bits + mode)
    codes = su.quantize(X)
    sc = su.score(Q, n, *codes)
    P.check_scores(su, sc, Q, *codes)


@pytest.mark.parametrize("nq", [1, 2, 3, 4, 6, 7, 8, 15])
def test_scores_every_pass_shape_and_determinism(nq):
    d = 264
    su = P.Setup(d, 4, tq.TQ_PROD)
    n = 1000
    X, Q = _data(d, n, nq, 77 + nq)
    codes = su.quantize(X)
    sc = su.score(Q, n, *codes)
    ref = P.check_scores(su, sc, Q, *codes)
    assert torch.equal(sc, su.score(Q, n, *codes))
    # a query's estimate does not depend on which other queries share its pass
    one = su.score(Q[nq - 1:nq].contiguous(), n, *codes)
    assert torch.equal(one[0], sc[nq - 1])
    ts, ti = su.topk(Q, n, *codes, 37)
    P.check_topk(ref, P.score_tolerance(su, Q, codes[3], n), ts, ti, 37)


@pytest.mark.parametrize("d,bits,mode", [(128, 1, tq.TQ_MSE), (200, 2, tq.TQ_MSE), (520, 3, tq.TQ_MSE), (264, 4, tq.TQ_MSE),
                                          (128, 1, tq.TQ_PROD), (200, 2, tq.TQ_PROD), (1536, 3, tq.TQ_PROD),
                                          (520, 4, tq.TQ_PROD), (264, 5, tq.TQ_PROD)])
def test_many_query_engine_every_bit_width(d, bits, mode):
    """Seven or more queries take the tcgen05 engine (32 queries per pass); its estimates equal the
    few-query engine's bit for bit, and both match the oracle."""
    su = P.Setup(d, bits, mode)
    n, nq = 700, 37
    X, Q = _data(d, n, nq, 31 * d + bits + mode)
    codes = su.quantize(X)
    sc = su.score(Q, n, *codes)
    P.check_scores(su, sc, Q, *codes)
    few = su.score(Q[:3].contiguous(), n, *codes)
    assert torch.equal(few, sc[:3])
    last = su.score(Q[nq - 2:].contiguous(), n, *codes)
    assert torch.equal(last, sc[nq - 2:])
    ts, ti = su.topk(Q, n, *codes, 25)
    for q in (0, 17, nq - 1):
        vals, order = torch.sort(sc[q], descending=True, stable=True)
        assert torch.equal(ti[q].long(), order[:25]) and torch.equal(ts[q], vals[:25])


def test_many_query_engine_groups_of_256_and_filter_flow():
    cfg = wl.CONFIGS["c2"]
    su = P.Setup(cfg.d, 3, tq.TQ_PROD, cfg.pi_seed, cfg.s_seed)
    n, nq, k = 66000, 300, 10            # two groups of B operands (256 + 44 queries), thresholded top-k
    X, Q = wl.database(cfg, n, device=DEV), wl.queries(cfg, nq, device=DEV)
    codes = su.quantize(X)
    sc = su.score(Q, n, *codes)
    ts, ti = su.topk(Q, n, *codes, k)
    for q in (0, 31, 32, 255, 256, 299):
        one = su.score(Q[q:q + 1].contiguous(), n, *codes)
        assert torch.equal(one[0], sc[q])
        vals, order = torch.sort(sc[q], descending=True, stable=True)
        assert torch.equal(ti[q].long(), order[:k]) and torch.equal(ts[q], vals[:k])
    P.check_scores(su, sc[:4, :2000].contiguous(), Q[:4].contiguous(), *(None if t is None else t[:2000].contiguous() for t in codes))


def test_zero_and_huge_queries_and_unit_norm_codes():
    d = 200
    su = P.Setup(d, 3, tq.TQ_PROD)
    n = 500
    X, Q = _data(d, n, 4, 5)
    Q[1].zero_()
    Q[2] *= 1e6
    Q[3] *= 1e-6
    idx, qjl, gamma, _ = su.quantize(torch.nn.functional.normalize(X, dim=1), with_norms=False)
    sc = su.score(Q, n, idx, qjl, gamma, None)
    P.check_scores(su, sc, Q, idx, qjl, gamma, None)
    assert bool((sc[1] == 0).all())


def test_topk_threshold_filter_flow_matches_oracle():
    cfg = wl.CONFIGS["c2"]
    su = P.Setup(cfg.d, 3, tq.TQ_PROD, cfg.pi_seed, cfg.s_seed)
    n, nq, k = 70001, 6, 100
    X, Q = wl.database(cfg, n, device=DEV), wl.queries(cfg, nq, device=DEV)
    codes = su.quantize(X)
    sc = su.score(Q, n, *codes)
    ref = P.check_scores(su, sc, Q, *codes)
    tol = P.score_tolerance(su, Q, codes[3], n)
    ts, ti = su.topk(Q, n, *codes, k)
    P.check_topk(ref, tol, ts, ti, k)
    # exactly the library's own dense scores, sorted (score desc, id asc)
    for q in range(nq):
        order = np.lexsort((np.arange(n), -sc[q].cpu().numpy().astype(np.float64)))[:k]
        assert np.array_equal(ti[q].cpu().numpy(), order)
        assert torch.equal(ts[q], sc[q][torch.from_numpy(order).to(DEV)])
    # the minimum workspace takes the dense block flow and must agree bit for bit
    small = tq.tq_workspace_bytes(su.plan, tq.TQ_OP_TOPK, 4096, nq, k)
    ts2, ti2 = su.topk(Q, n, *codes, k, workspace_bytes=small)
    assert torch.equal(ts, ts2) and torch.equal(ti, ti2)


def test_topk_overflow_rescue_on_massive_ties():
    """All vectors identical: every score ties, the candidate list overflows, the rescue pass must
    return the k smallest ids."""
    d = 128
    su = P.Setup(d, 2, tq.TQ_MSE)
    n, k = 66000, 50
    row = torch.randn((1, d), generator=torch.Generator().manual_seed(3))
    X = row.expand(n, d).contiguous().to(DEV)
    Q = torch.randn((2, d), generator=torch.Generator().manual_seed(4)).to(DEV)
    codes = su.quantize(X)
    ts, ti = su.topk(Q, n, *codes, k)
    assert torch.equal(ti, torch.arange(k, dtype=torch.int32, device=DEV).expand(2, k))
    sc = su.score(Q, n, *codes)
    assert torch.equal(ts, sc[:, :k])


def test_topk_adversarial_order_descending_scores():
    """Best vectors last: the pilot threshold is weak, the filter admits many candidates."""
    cfg = wl.CONFIGS["c2"]
    su = P.Setup(cfg.d, 3, tq.TQ_PROD, cfg.pi_seed, cfg.s_seed)
    n, k = 66049, 64
    X = wl.database(cfg, n, device=DEV)
    Q = wl.queries(cfg, 1, device=DEV)
    order = torch.argsort(X @ Q[0])            # ascending true inner product
    X = X[order].contiguous()
    codes = su.quantize(X)
    sc = su.score(Q, n, *codes)
    ts, ti = su.topk(Q, n, *codes, k)
    want = np.lexsort((np.arange(n), -sc[0].cpu().numpy().astype(np.float64)))[:k]
    assert np.array_equal(ti[0].cpu().numpy(), want)


_KERNEL_FORM_CHILD = r"""
import sys
import torch
sys.path.insert(0, sys.argv[1])
import paper_2504_19874_b200 as tq
from tests import parity as P
blob = torch.load(sys.argv[2])
for case in blob["cases"]:
    su = P.Setup(case["d"], case["bits"], case["mode"], layout=case["layout"])
    codes = tuple(None if t is None else t.to("cuda:0") for t in case["codes"])
    Q = case["Q"].to("cuda:0")
    n = case["n"]
    sc = su.score(Q, n, *codes)
    assert torch.equal(sc.cpu(), case["scores"]), "dense scores differ"
    ts, ti = su.topk(Q, n, *codes, case["k"])
    assert torch.equal(ts.cpu(), case["top_scores"]) and torch.equal(ti.cpu(), case["top_ids"]), "top-k differs"
print("kernel form ok")
"""


@pytest.mark.parametrize("env", [{"TQ_SCAN_WIDE": "0"}, {"TQ_SCAN_PAIRS": "0"}])
def test_other_forms_of_the_many_query_kernel_give_the_same_estimates(env, tmp_path):
    """Calls of more than 32 queries run the wide tcgen05 kernel (64 queries per pass) on CTA pairs.  TQ_SCAN_WIDE=0
    keeps the 32-query kernel and TQ_SCAN_PAIRS=0 runs the wide kernel on single CTAs (both read once per process): the
    same integers, so dense estimates and top-k must be bit-identical.  Sizes: an odd number of 128-vector tiles with a
    ragged tail, 70 queries (a full pass and a short one), and one thresholded top-k (n >= 65,536)."""
    import os
    import subprocess
    import sys
    cases = []
    for d, bits, mode, layout, n, k in ((1536, 4, tq.TQ_PROD, tq.TQ_LAYOUT_NIBBLE, 1300, 20), (264, 4, tq.TQ_PROD, None, 1300, 20),
                                        (520, 3, tq.TQ_MSE, None, 1300, 20), (200, 3, tq.TQ_PROD, None, 66000, 10)):
        su = P.Setup(d, bits, mode, layout=layout)
        X, Q = _data(d, n, 70, 7 * d + bits)
        codes = su.quantize(X)
        sc = su.score(Q, n, *codes)
        if n <= 2000:
            P.check_scores(su, sc, Q, *codes)
        ts, ti = su.topk(Q, n, *codes, k)
        cases.append({"d": d, "bits": bits, "mode": mode, "layout": layout, "n": n, "k": k, "Q": Q.cpu(),
                      "codes": tuple(None if t is None else t.cpu() for t in codes), "scores": sc.cpu(),
                      "top_scores": ts.cpu(), "top_ids": ti.cpu()})
    blob = tmp_path / "scan_forms.pt"
    torch.save({"cases": cases}, blob)
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-c", _KERNEL_FORM_CHILD, root, str(blob)], env=dict(os.environ, **env),
                       capture_output=True, text=True, timeout=900)
    assert r.returncode == 0 and "kernel form ok" in r.stdout, r.stdout[-2000:] + r.stderr[-2000:]


@pytest.mark.parametrize("nq", [33, 48, 49, 64, 65, 97])
@pytest.mark.parametrize("n", [1, 127, 129, 1153])
def test_wide_many_query_kernel_query_counts_and_ragged_tiles(nq, n):
    """More than 32 queries take the 64-query kernel: one query in the second half of a pass (33), a half-filled and a
    just-over-half second set (48, 49), a full pass (64), a full pass plus a 32-query-kernel pass of one (65) and 64 + 33
    (97); a single row, one ragged tile, one tile plus one row, and an odd number of tiles with a ragged tail.  Every
    query's row must equal what the few-query engine gives for it alone, and everything must match the oracle."""
    d = 264
    su = P.Setup(d, 4, tq.TQ_PROD)
    X, Q = _data(d, n, nq, 13 * nq + n)
    codes = su.quantize(X)
    sc = su.score(Q, n, *codes)
    P.check_scores(su, sc, Q, *codes)
    for q in (0, 31, 32, nq - 1):
        one = su.score(Q[q:q + 1].contiguous(), n, *codes)
        assert torch.equal(one[0], sc[q])
    k = min(n, 9)
    ts, ti = su.topk(Q, n, *codes, k)
    for q in (0, 32, nq - 1):
        vals, order = torch.sort(sc[q], descending=True, stable=True)
        assert torch.equal(ti[q].long(), order[:k]) and torch.equal(ts[q], vals[:k])


def test_wide_kernel_topk_overflow_rescue_and_adversarial_order():
    """The two hard top-k flows with 40 queries (the 64-query kernel in filter mode).  All vectors identical: every
    score ties, each CTA's shared-memory list and then the global candidate list overflow, and the guarded rescue pass
    must return the k smallest ids.  Best vectors last: the pilot threshold is weak and the filter admits many pairs."""
    d = 128
    su = P.Setup(d, 2, tq.TQ_MSE)
    n, k, nq = 66000, 50, 40
    row = torch.randn((1, d), generator=torch.Generator().manual_seed(3))
    X = row.expand(n, d).contiguous().to(DEV)
    Q = torch.randn((nq, d), generator=torch.Generator().manual_seed(4)).to(DEV)
    codes = su.quantize(X)
    ts, ti = su.topk(Q, n, *codes, k)
    assert torch.equal(ti, torch.arange(k, dtype=torch.int32, device=DEV).expand(nq, k))
    sc = su.score(Q, n, *codes)
    assert torch.equal(ts, sc[:, :k])

    cfg = wl.CONFIGS["c2"]
    su = P.Setup(cfg.d, 3, tq.TQ_PROD, cfg.pi_seed, cfg.s_seed)
    n, k = 66049, 64
    X = wl.database(cfg, n, device=DEV)
    Q = wl.queries(cfg, nq, device=DEV)
    order = torch.argsort(X @ Q[:8].mean(dim=0))     # ascending inner product with the first queries' mean
    X = X[order].contiguous()
    codes = su.quantize(X)
    sc = su.score(Q, n, *codes)
    ts, ti = su.topk(Q, n, *codes, k)
    for q in (0, 7, 33, nq - 1):
        want = np.lexsort((np.arange(n), -sc[q].cpu().numpy().astype(np.float64)))[:k]
        assert np.array_equal(ti[q].cpu().numpy(), want)
        assert torch.equal(ts[q], sc[q][torch.from_numpy(want).to(DEV)])
