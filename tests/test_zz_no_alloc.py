"""tq_score_static: scoring for callers that cannot allocate device memory.

Some users of this library must not call cudaMalloc while they score: a server that handed the whole
GPU to its own pool at start-up, a plug-in whose host forbids allocations after initialisation, a
real-time loop that cannot take the device-wide stall an allocation may cause.  For them the library
keeps the rotated-query workspace in an array of its own.  This test calls that entry point through
the C ABI twice in a row, with different queries, and checks each result against tq_score given an
ordinary caller workspace: the array is shared and keeps the previous call's contents, so the second
call would expose anything stale.  Both entry points run the same scan kernels on the same operands, so
the results must agree bit for bit; the free device memory must not move across the call.  The file
sorts last so that a run stopping at the first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

import paper_2504_19874_b200 as tq
import tq_workloads as wl
from tests import parity as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _score_both_ways(su, Q, n, codes):
    idx, qjl, gamma, norms = codes
    want = su.score(Q, n, idx, qjl, gamma, norms)                     # caller-provided workspace
    got = torch.full_like(want, float("nan"))
    tq.tq_score_static(su.plan, Q, n, idx, qjl, gamma, norms, got)    # library's built-in array
    torch.cuda.synchronize()
    first = got.clone()
    got.fill_(float("nan"))
    free_before = torch.cuda.mem_get_info()[0]                        # (code of every kernel involved is loaded by now)
    tq.tq_score_static(su.plan, Q, n, idx, qjl, gamma, norms, got)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before                # the call obtained no device memory
    assert torch.equal(first, got)
    tol = torch.from_numpy(P.score_tolerance(su, Q, norms, n)).to(want.device)
    tol = torch.maximum(tol, P.RTOL * want.abs().double())
    assert bool(((got.double() - want.double()).abs() <= tol).all())
    assert torch.equal(got, want)                                     # same kernels, same operands: same bits
    return want


def test_static_scratch_matches_workspace_variant_on_two_calls_in_a_row():
    cfg = wl.CONFIGS["c2"]
    su = P.Setup(cfg.d, 3, tq.TQ_PROD, cfg.pi_seed, cfg.s_seed)
    n = 3000
    X = wl.database(cfg, n, device=DEV)
    codes = su.quantize(X)
    Qa = wl.queries(cfg, 12, device=DEV)
    Qb = wl.make_vectors(cfg, 5, 777, DEV) * 3.0
    first = _score_both_ways(su, Qa, n, codes)
    second = _score_both_ways(su, Qb, n, codes)                       # fewer queries: leftovers of call 1 remain behind them
    assert not torch.equal(first[:5], second)
    # and against the oracle, like every other score test
    P.check_scores(su, second, Qb, *codes)


@pytest.mark.parametrize("d,bits,mode,layout,nq", [(64, 3, tq.TQ_PROD, None, 9), (1536, 4, tq.TQ_PROD, None, 40),
                                                   (1536, 4, tq.TQ_PROD, tq.TQ_LAYOUT_NIBBLE, 11),
                                                   (520, 2, tq.TQ_MSE, None, 3)])
def test_static_scratch_runs_the_engines_of_tq_score(d, bits, mode, layout, nq):
    """CUDA-core path (d < 128), both bit-plane engines (40 queries at d = 1536: the many-query engine's operand
    does not fit the array, the few-query engine takes over with the same estimates) and the nibble layout."""
    su = P.Setup(d, bits, mode, layout=layout)
    n = 900
    g = torch.Generator(device="cpu").manual_seed(d + nq)
    X = torch.randn((n, d), generator=g).to(DEV)
    codes = su.quantize(X)
    assert nq <= tq.tq_score_static_max_queries(su.plan)
    for scale in (1.0, 0.25):
        Q = (torch.randn((nq, d), generator=g) * scale).to(DEV)
        _score_both_ways(su, Q, n, codes)


def test_static_scratch_rejects_requests_beyond_its_size():
    d = 1536
    su = P.Setup(d, 2, tq.TQ_MSE)
    n = 64
    X = wl.database(wl.CONFIGS["c4"], n, device=DEV)
    codes = su.quantize(X)
    too_many = tq.tq_score_static_max_queries(su.plan) + 1
    assert 100 < too_many <= tq.TQ_STATIC_SCRATCH_BYTES // (d * 4) + 1
    Q = torch.randn((too_many, d), device=DEV)
    out = torch.zeros((too_many, n), device=DEV)
    with pytest.raises(tq.TqError) as e:
        tq.tq_score_static(su.plan, Q, n, *codes, out)
    assert e.value.code == 7 and "built-in array" in str(e.value)
    assert not bool(out.any())                                        # nothing was launched
    ok = Q[: too_many - 1].contiguous()
    _score_both_ways(su, ok, n, codes)
