"""TQ_LAYOUT_NIBBLE (TQ_PROD, b = 4): the layout itself against its written definition and the canonical bit
streams, and every consumer of the codes (scan engines in both operand shapes, top-k flows, dequantisation,
weighted sums) against the oracle on codes held in that layout."""
import numpy as np
import pytest
import torch

import paper_2504_19874_b200 as tq
import tq_workloads as wl
from oracle import turboquant_oracle as orc
from tests import parity as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
NIB = tq.TQ_LAYOUT_NIBBLE


def _data(d, n, nq, seed):
    g = torch.Generator(device="cpu").manual_seed(seed)
    X = (torch.randn((n, d), generator=g) * torch.rand((n, 1), generator=g).mul(2).add(0.3)).to(DEV)
    Q = (torch.randn((nq, d), generator=g) * torch.rand((nq, 1), generator=g).mul(4).add(0.1)).to(DEV)
    return X, Q


@pytest.mark.parametrize("d", [128, 200, 264, 520, 1536])
def test_layout_is_a_permutation_of_the_canonical_codes(d):
    n = 300
    X, _ = _data(d, n, 1, 11 * d)
    can = P.Setup(d, 4, tq.TQ_PROD)
    nib = P.Setup(d, 4, tq.TQ_PROD, layout=NIB)
    assert nib.plan.layout == NIB and can.plan.layout == tq.TQ_LAYOUT_CANONICAL
    idx_c, qjl_c, gamma_c, norms_c = can.quantize(X)
    idx_n, qjl_n, gamma_n, norms_n = nib.quantize(X)
    assert torch.equal(gamma_c, gamma_n) and torch.equal(norms_c, norms_n)
    # the definition, read by numpy: same indices and sign bits, unused nibbles zero
    i3, bit, rest = P.nibble_rows_to_coordinates(idx_n.cpu().numpy(), qjl_n.cpu().numpy(), d)
    assert not rest.any()
    assert np.array_equal(i3, orc.unpack_bits(idx_c.cpu().numpy(), 3, d))
    assert np.array_equal(bit, orc.unpack_bits(qjl_c.cpu().numpy(), 1, d))
    # the library's converter, both ways, in place
    a, b = idx_c.clone(), qjl_c.clone()
    tq.tq_convert_layout(can.plan, n, a, b, tq.TQ_LAYOUT_CANONICAL, NIB)
    assert torch.equal(a, idx_n) and torch.equal(b, qjl_n)
    tq.tq_convert_layout(can.plan, n, a, b, NIB, tq.TQ_LAYOUT_CANONICAL)
    assert torch.equal(a, idx_c) and torch.equal(b, qjl_c)
    # and the codes against the oracle
    P.check_quantize(nib, X, idx_n, qjl_n, gamma_n, norms_n)


def test_layout_is_refused_where_it_does_not_exist():
    for d, bits, mode in ((64, 4, tq.TQ_PROD), (256, 3, tq.TQ_PROD), (256, 3, tq.TQ_MSE), (256, 5, tq.TQ_PROD)):
        su = P.Setup(d, bits, mode)
        with pytest.raises(tq.TqError) as e:
            su.plan.set_layout(NIB)
        assert e.value.code == 2
        assert su.plan.layout == tq.TQ_LAYOUT_CANONICAL


@pytest.mark.parametrize("d", [128, 200, 520, 1536, 3072])
@pytest.mark.parametrize("nq", [1, 2, 3, 8, 11, 37])
def test_scores_every_engine_and_operand_shape(d, nq):
    su = P.Setup(d, 4, tq.TQ_PROD, layout=NIB)
    n = 300 if d >= 1536 else 777
    X, Q = _data(d, n, nq, 1000 * d + nq)
    codes = su.quantize(X)
    sc = su.score(Q, n, *codes)
    P.check_scores(su, sc, Q, *codes)
    assert torch.equal(sc, su.score(Q, n, *codes))
    # a query's estimate does not depend on which other queries share its pass, nor on the operand shape or engine
    # (two-query and eight-query register-fed shapes, tcgen05 with 32 queries per pass)
    one = su.score(Q[nq - 1:nq].contiguous(), n, *codes)
    assert torch.equal(one[0], sc[nq - 1])
    if nq > 8:
        assert torch.equal(su.score(Q[:8].contiguous(), n, *codes), sc[:8])


def test_measured_error_of_both_engines():
    """Worst |estimate - oracle| in units of ||q|| ||x|| for the bit-plane engine on canonical codes and the
    table-lookup engine on nibble codes (the 16-bit centroid table and the two-digit sign-bit weights of the
    latter are its only extra rounding): both far inside the 1e-4 of the parity rule."""
    d, n = 1536, 1000
    X, Q = _data(d, n, 4, 5)
    worst = {}
    for name, layout in (("canonical", None), ("nibble", NIB)):
        su = P.Setup(d, 4, tq.TQ_PROD, layout=layout)
        codes = su.quantize(X)
        ref = P.check_scores(su, su.score(Q, n, *codes), Q, *codes)
        got = P.as_f64(su.score(Q, n, *codes))
        scale = np.linalg.norm(P.as_f64(Q), axis=1)[:, None] * np.linalg.norm(P.as_f64(X), axis=1)[None, :]
        worst[name] = float((np.abs(got - ref) / scale).max())
    print("worst score error / (||q|| ||x||):", worst)
    assert worst["canonical"] < 2e-5 and worst["nibble"] < 3e-6


def test_zero_huge_and_tiny_queries():
    d, n = 200, 500
    su = P.Setup(d, 4, tq.TQ_PROD, layout=NIB)
    X, Q = _data(d, n, 4, 6)
    Q[1].zero_()
    Q[2] *= 1e6
    Q[3] *= 1e-6
    codes = su.quantize(X)
    sc = su.score(Q, n, *codes)
    P.check_scores(su, sc, Q, *codes)
    assert bool((sc[1] == 0).all())


def test_topk_flows():
    cfg = wl.CONFIGS["c4"]
    d = 264
    su = P.Setup(d, 4, tq.TQ_PROD, layout=NIB)
    n, k = 70001, 100
    for nq in (2, 6, 19, 40):
        X, Q = _data(d, n, nq, 99 + nq)
        codes = su.quantize(X)
        sc = su.score(Q, n, *codes)
        ts, ti = su.topk(Q, n, *codes, k)
        for q in range(nq):
            order = np.lexsort((np.arange(n), -sc[q].cpu().numpy().astype(np.float64)))[:k]
            assert np.array_equal(ti[q].cpu().numpy(), order)
            assert torch.equal(ts[q], sc[q][torch.from_numpy(order).to(DEV)])
        small = tq.tq_workspace_bytes(su.plan, tq.TQ_OP_TOPK, 4096, nq, k)
        ts2, ti2 = su.topk(Q, n, *codes, k, workspace_bytes=small)
        assert torch.equal(ts, ts2) and torch.equal(ti, ti2)
    ref = P.check_scores(su, sc[:, :3000].contiguous(), Q, *(t[:3000].contiguous() for t in codes))
    ts, ti = su.topk(Q, 3000, *(t[:3000].contiguous() for t in codes), 37)
    P.check_topk(ref, P.score_tolerance(su, Q, codes[3][:3000], 3000), ts, ti, 37)
    del cfg


def test_dequantize_and_weighted_sum():
    d, n = 200, 1500
    su = P.Setup(d, 4, tq.TQ_PROD, layout=NIB)
    X, _ = _data(d, n, 1, 8)
    codes = su.quantize(X)
    Xh = su.dequantize(n, *codes)
    ref = P.check_dequant(su, Xh, *codes)
    g = torch.Generator(device="cpu").manual_seed(3)
    W = torch.rand((3, n), generator=g).to(DEV)
    out = torch.empty((3, d), device=DEV)
    ws = torch.empty(tq.tq_workspace_bytes(su.plan, tq.TQ_OP_WSUM, n, 3), dtype=torch.uint8, device=DEV)
    tq.tq_wsum(su.plan, W, n, *codes, out, ws)
    want = P.as_f64(W) @ ref
    err = np.linalg.norm(P.as_f64(out) - want, axis=1) / np.linalg.norm(want, axis=1)
    assert float(err.max()) < 1e-4
