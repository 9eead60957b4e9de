"""Parity at the full sizes of the evaluation configurations, in the launch configuration the benchmark
times (default scratch / workspace sizes): the oracle checks sampled vectors one by one, and properties
that hold at any size cover the rest (the thresholded top-k equals the sort of the library's own dense
scores; no unsampled vector beats the k-th)."""
import numpy as np
import pytest
import torch

import paper_2504_19874_b200 as tq
import tq_workloads as wl
from tests import parity as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _sample_rows(n, count, seed):
    g = torch.Generator(device="cpu").manual_seed(seed)
    rows = torch.randperm(n, generator=g)[:count].sort().values
    # always include the first and last rows and a block boundary of the quantiser
    extra = torch.tensor([0, 1, 65535, 65536, n - 1])
    return torch.unique(torch.cat([rows, extra[extra < n]])).to(DEV)


def _check_full(name, bits, mode, n, nq, k, samples=1536, layout=None):
    cfg = wl.CONFIGS[name]
    su = P.Setup(cfg.d, bits, mode, cfg.pi_seed, cfg.s_seed, layout=layout)
    X = wl.database(cfg, n, device=DEV)
    Q = wl.queries(cfg, nq, device=DEV)
    idx, qjl, gamma, norms = su.quantize(X)
    rows = _sample_rows(n, samples, 17)
    sub = lambda t: None if t is None else t[rows].contiguous()
    stats = P.check_quantize(su, X[rows].contiguous(), sub(idx), sub(qjl), sub(gamma), sub(norms))
    assert stats["idx_mismatch"] == 0 and stats.get("qjl_mismatch", 0) <= P.MAX_MISMATCH
    del X
    # scores of the sampled vectors against the oracle, through the full-size launch
    sc = su.score(Q, n, idx, qjl, gamma, norms)
    ref = P.check_scores(su, sc[:, rows].contiguous(), Q, sub(idx), sub(qjl), sub(gamma), sub(norms))
    # top-k: identical to sorting the library's dense scores (score desc, id asc) ...
    ts, ti = su.topk(Q, n, idx, qjl, gamma, norms, k)
    for q in range(nq):
        row = sc[q]
        vals, order = torch.sort(row, descending=True, stable=True)
        assert torch.equal(ti[q].long(), order[:k]) and torch.equal(ts[q], vals[:k])
    # ... whose returned entries the oracle confirms one by one
    for q in range(min(nq, 4)):
        ids = ti[q].long()
        codes_q = tuple(None if t is None else t[ids].contiguous() for t in (idx, qjl, gamma, norms))
        P.check_scores(su, ts[q:q + 1].contiguous(), Q[q:q + 1].contiguous(), *codes_q)
        tol = P.score_tolerance(su, Q[q:q + 1], sub(norms), rows.numel())
        outside = ~torch.isin(rows, ids).cpu().numpy()                   # sampled vectors that were not returned
        assert np.all(ref[q][outside] <= float(ts[q, -1]) + 2 * tol[0][outside])   # none of them beats the k-th
    return stats


def test_c4_d1536_prod_b4_one_million():
    _check_full("c4", 4, tq.TQ_PROD, 1_000_000, 8, 100)


def test_c4_d1536_prod_b4_one_million_nibble_layout():
    _check_full("c4", 4, tq.TQ_PROD, 1_000_000, 8, 100, layout=tq.TQ_LAYOUT_NIBBLE)


def test_c4_d1536_prod_b4_one_million_nibble_layout_many_queries():
    """96 queries: a full pass of the 64-query tcgen05 kernel and a pass of the 32-query kernel, dense and thresholded,
    in the launch configuration of the benchmark's many-query leg."""
    _check_full("c4", 4, tq.TQ_PROD, 1_000_000, 96, 100, layout=tq.TQ_LAYOUT_NIBBLE)


def test_c4_d1536_mse_b2_one_million():
    _check_full("c4", 2, tq.TQ_MSE, 1_000_000, 8, 100)


def test_c2_d200_prod_b3_one_million():
    _check_full("c2", 3, tq.TQ_PROD, 1_000_000, 64, 100)


@pytest.mark.parametrize("bits,k", [(2, 10), (4, 100)])
def test_c5_d3072_prod(bits, k):
    _check_full("c5", bits, tq.TQ_PROD, 1_000_000, 8, k, samples=768, layout=tq.TQ_LAYOUT_NIBBLE if bits == 4 else None)
