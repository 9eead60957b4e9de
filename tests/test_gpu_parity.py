"""GPU-vs-oracle parity through the C ABI (needs a B200).  Same seeded inputs on both sides."""
import numpy as np
import pytest
import torch

import paper_2504_19874_b200 as tq
import tq_workloads as wl
from oracle import turboquant_oracle as orc
from tests import parity as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run_case(su, X, Q, k=None, with_norms=True, unit_input=False):
    n = X.shape[0]
    idx, qjl, gamma, norms = su.quantize(X, with_norms=with_norms)
    stats = P.check_quantize(su, X, idx, qjl, gamma, norms, unit_input=unit_input)
    Xh = su.dequantize(n, idx, qjl, gamma, norms)
    P.check_dequant(su, Xh, idx, qjl, gamma, norms)
    if Q is not None:
        sc = su.score(Q, n, idx, qjl, gamma, norms)
        ref = P.check_scores(su, sc, Q, idx, qjl, gamma, norms)
        if k:
            ts, ti = su.topk(Q, n, idx, qjl, gamma, norms, k)
            P.check_topk(ref, P.score_tolerance(su, Q, norms, n), ts, ti, k)
    return stats


def test_config1_mse_d128_b2_full():
    cfg = wl.CONFIGS["c1"]
    su = P.Setup(cfg.d, 2, tq.TQ_MSE, cfg.pi_seed, cfg.s_seed)
    X, Q = wl.database(cfg, device=DEV), wl.queries(cfg, device=DEV)
    stats = run_case(su, X, Q, k=10)
    assert stats["idx_mismatch"] == 0


@pytest.mark.parametrize("d,bits,mode,n", [
    (8, 1, tq.TQ_MSE, 1), (8, 2, tq.TQ_PROD, 127), (16, 3, tq.TQ_MSE, 129), (16, 4, tq.TQ_PROD, 300),
    (64, 3, tq.TQ_PROD, 1000), (64, 2, tq.TQ_PROD, 777), (64, 3, tq.TQ_MSE, 513), (64, 2, tq.TQ_MSE, 64),
    (200, 3, tq.TQ_PROD, 1500), (200, 4, tq.TQ_MSE, 333), (40, 3, tq.TQ_MSE, 50), (24, 5, tq.TQ_PROD, 90),
    (128, 1, tq.TQ_PROD, 200), (128, 1, tq.TQ_MSE, 200), (264, 2, tq.TQ_PROD, 260),
])
def test_small_shapes_ragged_tails(d, bits, mode, n):
    su = P.Setup(d, bits, mode)
    g = torch.Generator(device="cpu").manual_seed(d * 100 + bits)
    X = (torch.randn((n, d), generator=g) * torch.rand((n, 1), generator=g).mul(3).add(0.2)).to(DEV)
    Q = torch.randn((5, d), generator=g).to(DEV)
    run_case(su, X, Q, k=min(7, n))


def test_many_query_path_and_topk_blocks():
    """nq above the few-query limit takes the tiled path; a small workspace forces several top-k blocks."""
    cfg = wl.CONFIGS["c2"]
    su = P.Setup(cfg.d, 3, tq.TQ_PROD, cfg.pi_seed, cfg.s_seed)
    n, nq, k = 20000, 40, 100
    X, Q = wl.database(cfg, n, device=DEV), wl.queries(cfg, nq, device=DEV)
    idx, qjl, gamma, norms = su.quantize(X)
    P.check_quantize(su, X, idx, qjl, gamma, norms)
    sc = su.score(Q, n, idx, qjl, gamma, norms)
    ref = P.check_scores(su, sc, Q, idx, qjl, gamma, norms)
    tol = P.score_tolerance(su, Q, norms, n)
    ts, ti = su.topk(Q, n, idx, qjl, gamma, norms, k)
    P.check_topk(ref, tol, ts, ti, k)
    small = tq.tq_workspace_bytes(su.plan, tq.TQ_OP_TOPK, 4096, nq, k)      # the documented minimum
    assert small < tq.tq_workspace_bytes(su.plan, tq.TQ_OP_TOPK, n, nq, k)
    ts2, ti2 = su.topk(Q, n, idx, qjl, gamma, norms, k, workspace_bytes=small)
    assert torch.equal(ts, ts2) and torch.equal(ti, ti2)
    # few-query path gives the same answers
    ts3, ti3 = su.topk(Q[:3].contiguous(), n, idx, qjl, gamma, norms, k)
    P.check_topk(ref[:3], tol[:3], ts3, ti3, k)


@pytest.mark.parametrize("name,bits,mode,n", [("c4", 4, tq.TQ_PROD, 2500), ("c4", 2, tq.TQ_MSE, 1300),
                                               ("c5", 2, tq.TQ_PROD, 700), ("c5", 4, tq.TQ_PROD, 600)])
def test_embedding_configs_subset(name, bits, mode, n):
    cfg = wl.CONFIGS[name]
    su = P.Setup(cfg.d, bits, mode, cfg.pi_seed, cfg.s_seed)
    X, Q = wl.database(cfg, n, device=DEV), wl.queries(cfg, 8, device=DEV)
    stats = run_case(su, X, Q, k=100)
    assert stats["idx_mismatch"] == 0


_ONE_CTA_CHILD = r"""
import sys, torch
sys.path.insert(0, sys.argv[1])
import paper_2504_19874_b200 as tq
import tq_workloads as wl
from tests import parity as P
blob = torch.load(sys.argv[2])
cfg = wl.CONFIGS["c4"]
for (bits, mode), want in zip(((4, tq.TQ_PROD), (2, tq.TQ_MSE)), blob["codes"]):
    su = P.Setup(cfg.d, bits, mode, cfg.pi_seed, cfg.s_seed)
    X = blob["X"].cuda()
    got = su.quantize(X)
    P.check_quantize(su, X, *got)
    for u, v in zip(got, want):
        assert (u is None and v is None) or torch.equal(u.cpu(), v), "the two GEMM kernels disagree"
print("one-CTA kernel ok")
"""


def test_one_cta_gemm_kernel_gives_the_same_codes(tmp_path):
    """Blocks of more than 128 rows run the quantiser's GEMMs on CTA pairs; TQ_GEMM_PAIRS=0 (read once per process)
    keeps the one-CTA kernel.  Same operands, same order of accumulation: the codes must be bit-identical, and the
    child checks them against the oracle as well."""
    import os
    import subprocess
    import sys
    cfg = wl.CONFIGS["c4"]
    X = wl.database(cfg, 1500, device=DEV)
    codes = []
    for bits, mode in ((4, tq.TQ_PROD), (2, tq.TQ_MSE)):
        su = P.Setup(cfg.d, bits, mode, cfg.pi_seed, cfg.s_seed)
        codes.append(tuple(None if t is None else t.cpu() for t in su.quantize(X)))
    blob = tmp_path / "pair_codes.pt"
    torch.save({"X": X.cpu(), "codes": codes}, blob)
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, TQ_GEMM_PAIRS="0")
    r = subprocess.run([sys.executable, "-c", _ONE_CTA_CHILD, root, str(blob)], env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "one-CTA kernel ok" in r.stdout, r.stdout[-2000:] + r.stderr[-2000:]


def test_small_scratch_forces_several_blocks_of_rows():
    cfg = wl.CONFIGS["c2"]
    for bits, mode in ((3, tq.TQ_PROD), (2, tq.TQ_MSE)):
        su = P.Setup(cfg.d, bits, mode, cfg.pi_seed, cfg.s_seed)
        X = wl.database(cfg, 1000, device=DEV)
        full = su.quantize(X)
        small = tq.tq_workspace_bytes(su.plan, tq.TQ_OP_QUANTIZE, 256)
        assert small < tq.tq_workspace_bytes(su.plan, tq.TQ_OP_QUANTIZE, 1000)
        part = su.quantize(X, scratch_bytes=small)
        for u, v in zip(full, part):
            assert (u is None and v is None) or torch.equal(u, v)
        P.check_quantize(su, X, *part)
        # a scratch between the minimum and the preferred size: more, smaller launches, same codes
        dpad = (cfg.d + 7) // 8 * 8
        piped = su.quantize(X, scratch_bytes=small + 256 * dpad * 4)
        for u, v in zip(full, piped):
            assert (u is None and v is None) or torch.equal(u, v)


@pytest.mark.parametrize("d", [64, 256])
def test_bf16_inputs_and_unit_norm_mode(d):
    su = P.Setup(d, 3, tq.TQ_PROD)
    g = torch.Generator(device="cpu").manual_seed(9)
    X = torch.randn((900, d), generator=g).to(torch.bfloat16).to(DEV)
    Q = torch.randn((4, d), generator=g).to(torch.bfloat16).to(DEV)
    run_case(su, X, Q, k=5)
    U = torch.nn.functional.normalize(torch.randn((400, d), generator=g), dim=1).to(DEV)
    run_case(su, U, Q, with_norms=False, unit_input=True)


def test_strided_rows_zero_vector_and_empty_input():
    d = 128
    su = P.Setup(d, 3, tq.TQ_PROD)
    g = torch.Generator(device="cpu").manual_seed(4)
    big = torch.randn((300, d + 32), generator=g).to(DEV)
    X = big[:, :d]
    X[17].zero_()
    assert X.stride(0) == d + 32
    idx, qjl, gamma, norms = su.quantize(X)
    P.check_quantize(su, X, idx, qjl, gamma, norms)
    assert norms[17].item() == 0 and gamma[17].item() == 0
    assert bool((qjl[17] == 0xFF).all())
    mid = (1 << (su.mse_bits - 1)) - 1
    assert np.all(orc.unpack_bits(idx[17:18].cpu().numpy(), su.mse_bits, d) == mid)
    Xh = su.dequantize(300, idx, qjl, gamma, norms)
    assert bool((Xh[17] == 0).all())
    # n = 0 is a no-op
    empty = torch.empty((0, d), device=DEV)
    tq.tq_quantize_prod(su.plan, empty, idx, qjl, gamma, norms, None)


def test_determinism_and_untouched_neighbours():
    d, n = 200, 1000
    su = P.Setup(d, 3, tq.TQ_PROD)
    X = wl.database(wl.CONFIGS["c2"], n, device=DEV)
    a = su.quantize(X)
    b = su.quantize(X)
    for u, v in zip(a, b):
        assert torch.equal(u, v)
    # guard rows around the outputs stay untouched
    rb = su.idx_rb
    buf = torch.full((n + 2, rb), 0x5A, dtype=torch.uint8, device=DEV)
    qb = torch.full((n + 2, su.qjl_rb), 0x5A, dtype=torch.uint8, device=DEV)
    gm = torch.full((n + 2,), 123.0, device=DEV)
    nm = torch.full((n + 2,), 123.0, device=DEV)
    ws = torch.empty(tq.tq_workspace_bytes(su.plan, tq.TQ_OP_QUANTIZE, n), dtype=torch.uint8, device=DEV)
    tq.tq_quantize_prod(su.plan, X, buf[1:-1], qb[1:-1], gm[1:-1], nm[1:-1], ws)
    torch.cuda.synchronize()
    for t in (buf, qb):
        assert bool((t[0] == 0x5A).all()) and bool((t[-1] == 0x5A).all())
    assert gm[0] == 123 and gm[-1] == 123 and nm[0] == 123 and nm[-1] == 123
    assert torch.equal(buf[1:-1], a[0]) and torch.equal(qb[1:-1], a[1])


def test_argument_errors_on_device():
    d = 64
    su = P.Setup(d, 3, tq.TQ_PROD)
    X = torch.randn((10, d), device=DEV)
    idx, qjl, gamma, norms = su.quantize(X)
    with pytest.raises(tq.TqError) as e:
        tq.tq_quantize_prod(su.plan, X, idx, qjl, gamma, norms, None)            # no scratch
    assert e.value.code == 7
    with pytest.raises(tq.TqError) as e:
        tq.tq_quantize_mse(su.plan, X, idx, norms)                                # wrong plan mode
    assert e.value.code == 1
    off = torch.empty(10 * su.idx_rb + 1, dtype=torch.uint8, device=DEV)[1:].view(10, su.idx_rb)
    ws = torch.empty(1 << 20, dtype=torch.uint8, device=DEV)
    with pytest.raises(tq.TqError) as e:
        tq.tq_quantize_prod(su.plan, X, off, qjl, gamma, norms, ws)               # misaligned idx
    assert e.value.code == 3
    ts = torch.empty((1, 20), device=DEV)
    ti = torch.empty((1, 20), dtype=torch.int32, device=DEV)
    with pytest.raises(tq.TqError) as e:
        tq.tq_topk(su.plan, X[:1], 10, idx, qjl, gamma, norms, 20, ts, ti, ws)   # k > n
    assert e.value.code == 2


def test_library_codebook_and_rotation_drive_the_same_path():
    """A plan built from the library's own set-up routines behaves like one built from the oracle's."""
    d = 128
    c, _ = tq.tq_codebook(d, 2)
    Pi = tq.tq_rotation(d, 52)
    su = P.Setup(d, 2, tq.TQ_MSE, 52, 53)
    assert np.array_equal(c, su.c)
    plan = tq.Plan(d, 2, tq.TQ_MSE, Pi, None, c)
    X = wl.database(wl.CONFIGS["c1"], 512, device=DEV)
    i1 = torch.empty((512, su.idx_rb), dtype=torch.uint8, device=DEV)
    n1 = torch.empty(512, device=DEV)
    sc = torch.empty(tq.tq_workspace_bytes(plan, tq.TQ_OP_QUANTIZE, 512), dtype=torch.uint8, device=DEV)
    tq.tq_quantize_mse(plan, X, i1, n1, sc)
    i2, _, _, n2 = su.quantize(X)
    assert (i1 != i2).float().mean().item() < 1e-3       # Pi differs by float32 rounding only
