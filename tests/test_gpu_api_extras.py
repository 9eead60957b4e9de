"""Entry points beside the seven of the hot path: prepared queries, the merge step of a sharded search
(tq_select_topk) and the bounded-wait self test."""
import numpy as np
import pytest
import torch

import paper_2504_19874_b200 as tq
from oracle import turboquant_oracle as orc
from tests import parity as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("d,bits,mode,layout,nq", [(64, 3, tq.TQ_PROD, None, 5), (264, 4, tq.TQ_PROD, None, 3),
                                                   (264, 4, tq.TQ_PROD, None, 41), (264, 2, tq.TQ_MSE, None, 300),
                                                   (264, 4, tq.TQ_PROD, tq.TQ_LAYOUT_NIBBLE, 2),
                                                   (1536, 4, tq.TQ_PROD, tq.TQ_LAYOUT_NIBBLE, 19)])
def test_prepared_queries_give_the_scores_of_tq_score(d, bits, mode, layout, nq):
    su = P.Setup(d, bits, mode, layout=layout)
    g = torch.Generator(device="cpu").manual_seed(7 * d + nq)
    n = 1100
    X = torch.randn((n, d), generator=g).to(DEV)
    Q = torch.randn((nq, d), generator=g).to(DEV)
    codes = su.quantize(X)
    want = su.score(Q, n, *codes)
    prepared = torch.empty(tq.tq_query_bytes(su.plan, nq), dtype=torch.uint8, device=DEV)
    tq.tq_query_prepare(su.plan, Q, prepared)
    for rows in (n, 257):          # the same prepared queries against two "segments"
        got = torch.full((nq, rows), float("nan"), device=DEV)
        tq.tq_score_prepared(su.plan, prepared, nq, rows, *(None if t is None else t[:rows].contiguous() for t in codes), got)
        torch.cuda.synchronize()
        assert torch.equal(got, want[:, :rows])
    with pytest.raises(tq.TqError) as e:
        tq.tq_query_prepare(su.plan, Q, prepared[:256])
    assert e.value.code == 7


def _select(cs, ci, k):
    nq = cs.shape[0]
    ts = torch.empty((nq, k), device=DEV)
    ti = torch.empty((nq, k), dtype=torch.int32, device=DEV)
    tq.tq_select_topk(cs, ci, k, ts, ti)
    torch.cuda.synchronize()
    return ts, ti


def _oracle_merge(cs, ci, k):
    """orc.topk over the valid pairs of each row, ordered by id so that its "lower position wins a tie" is
    "lower id wins"; missing entries are (-inf, -1)."""
    cs, ci = cs.cpu().numpy().astype(np.float64), ci.cpu().numpy()
    vals = np.full((cs.shape[0], k), -np.inf)
    ids = np.full((cs.shape[0], k), -1, dtype=np.int64)
    for q in range(cs.shape[0]):
        keep = np.nonzero(ci[q] >= 0)[0]
        keep = keep[np.argsort(ci[q][keep], kind="stable")]
        kk = min(k, keep.size)
        if kk:
            v, pos = orc.topk(cs[q][keep][None, :], kk)
            vals[q, :kk], ids[q, :kk] = v[0], ci[q][keep][pos[0]]
    return vals, ids


@pytest.mark.parametrize("m,k", [(8 * 1024, 1024), (8 * 100, 100), (50, 100), (1, 1), (20000, 7), (3000, 1)])
def test_select_topk_merges_like_the_oracle(m, k):
    g = torch.Generator(device="cpu").manual_seed(m + k)
    nq = 5
    # few distinct score values: many exact ties, also between "shards" (positions far apart)
    cs = (torch.randint(0, max(m // 8, 2), (nq, m), generator=g).float() / 7.0 - 3.0)
    ci = torch.stack([torch.randperm(4 * m + 11, generator=g)[:m] for _ in range(nq)]).int()
    empty = torch.rand((nq, m), generator=g) < 0.15
    ci[empty] = -1 - torch.randint(0, 5, (int(empty.sum()),), generator=g).int()   # empty slots: any negative id
    cs[0, :] = 1.5                                                                 # one query where everything ties
    ld = m + 13                                                                    # row stride larger than m
    buf_s = torch.full((nq, ld), float("inf"))
    buf_i = torch.full((nq, ld), 7, dtype=torch.int32)
    buf_s[:, :m], buf_i[:, :m] = cs, ci
    ts, ti = _select(buf_s.to(DEV)[:, :m], buf_i.to(DEV)[:, :m], k)
    want_s, want_i = _oracle_merge(cs, ci, k)
    assert np.array_equal(ti.cpu().numpy().astype(np.int64), want_i)
    assert np.array_equal(ts.cpu().numpy().astype(np.float64), want_s)


def test_select_topk_of_sharded_searches_equals_the_unsharded_search():
    d, n, nq, k, shards = 264, 30000, 6, 50, 3
    su = P.Setup(d, 3, tq.TQ_PROD)
    g = torch.Generator(device="cpu").manual_seed(12)
    X = torch.randn((n, d), generator=g)
    X[20001] = X[5]                      # equal vectors in different shards: equal scores, the lower id must win
    X[29999] = X[10000]
    X, Q = X.to(DEV), torch.randn((nq, d), generator=g).to(DEV)
    codes = su.quantize(X)
    whole_s, whole_i = su.topk(Q, n, *codes, k)
    cand_s, cand_i = [], []
    bounds = [0, 9000, 21000, n]
    for lo, hi in zip(bounds, bounds[1:]):
        part = tuple(None if t is None else t[lo:hi].contiguous() for t in codes)
        s, i = su.topk(Q, hi - lo, *part, k)
        cand_s.append(s)
        cand_i.append(i + lo)
    ts, ti = _select(torch.cat(cand_s, dim=1).contiguous(), torch.cat(cand_i, dim=1).contiguous(), k)
    assert torch.equal(ti, whole_i) and torch.equal(ts, whole_s)
    del shards


def test_bounded_wait_gives_up_and_reports_timeout():
    """A wait on a barrier nobody arrives at must end by itself after its limit, and the plan must report
    TQ_ERR_TIMEOUT once; the plan and the context stay usable."""
    su = P.Setup(128, 2, tq.TQ_MSE)
    tq.tq_plan_status(su.plan)                       # clean to begin with
    tq.tq_selftest_wait_timeout(su.plan, 20000)
    with pytest.raises(tq.TqError) as e:
        tq.tq_plan_status(su.plan)
    assert e.value.code == 6
    tq.tq_plan_status(su.plan)                       # the status was cleared by the report
    X = torch.randn((300, 128), generator=torch.Generator().manual_seed(1)).to(DEV)
    codes = su.quantize(X)                           # the context still works
    P.check_quantize(su, X, *codes)
