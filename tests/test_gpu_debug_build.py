"""The TQ_DEBUG build of the library (libtq_debug.so: every index check of the kernels' global stores and of the
caller's channel lists is compiled in) runs the hot path with the same results and a clean status, and turns an
index outside its array into TQ_ERR_BOUNDS without touching the memory.  Runs in a child process, because the
library variant is chosen when the binding loads."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

_CHILD = r"""
import math, sys
sys.path.insert(0, sys.argv[1])
import numpy as np, torch
import paper_2504_19874_b200 as tq
import paper_2504_19874_b200.binding as B
import tq_workloads as wl
from tests import parity as P
assert B._LIB_PATH.endswith("libtq_debug.so"), B._LIB_PATH
DEV = "cuda:0"
# quantise, scores, top-k on the tensor-core kernels (d = 256: pair GEMMs; nibble layout at b = 4)
for d, bits, mode, layout in ((256, 4, tq.TQ_PROD, tq.TQ_LAYOUT_NIBBLE), (256, 2, tq.TQ_MSE, None), (64, 3, tq.TQ_PROD, None)):
    su = P.Setup(d, bits, mode, layout=layout)
    g = torch.Generator(device="cpu").manual_seed(d + bits)
    X = torch.randn((3000, d), generator=g).to(DEV)
    Q = torch.randn((40, d), generator=g).to(DEV)
    codes = su.quantize(X)
    P.check_quantize(su, X, *codes)
    for nq in (1, 8, 40):
        sc = su.score(Q[:nq].contiguous(), 3000, *codes)
        P.check_scores(su, sc, Q[:nq].contiguous(), *codes)
    su.topk(Q[:8].contiguous(), 3000, *codes, 10)
    tq.tq_plan_status(su.plan)          # raises on any recorded status
# fused decode attention, then the same call with a channel index outside the output row
GROUP, HD = 64, 128
gK = (P.Setup(GROUP, 3, tq.TQ_PROD, 72, 73), P.Setup(GROUP, 2, tq.TQ_PROD, 74, 75))
gV = (P.Setup(GROUP, 3, tq.TQ_MSE, 76, 77), P.Setup(GROUP, 2, tq.TQ_MSE, 78, 79))
heads, T, qpk = 2, 700, 4
K, V, Q = wl.kv_cache(heads=heads, tokens=T, q_per_kv=qpk, seed=4, device=DEV)
groups = []
for gi in range(2):
    ch = torch.arange(gi * GROUP, (gi + 1) * GROUP, device=DEV)
    ck = [gK[gi].quantize(K[h][:, ch].float().contiguous()) for h in range(heads)]
    cv = [gV[gi].quantize(V[h][:, ch].float().contiguous()) for h in range(heads)]
    cat = lambda cs, i: torch.cat([c[i] for c in cs]).contiguous()
    groups.append({"plan_k": gK[gi].plan, "plan_v": gV[gi].plan, "k_idx": cat(ck, 0), "k_qjl": cat(ck, 1), "k_gamma": cat(ck, 2),
                   "k_norms": cat(ck, 3), "v_idx": cat(cv, 0), "v_norms": cat(cv, 3),
                   "k_channels": ch.to(torch.int32).repeat(heads, 1).contiguous(), "v_channels": ch.to(torch.int32).repeat(heads, 1).contiguous()})
ws = torch.empty(tq.tq_attend_decode_workspace_bytes(2, heads, T, GROUP), dtype=torch.uint8, device=DEV)
out = torch.zeros((heads * qpk, HD), device=DEV)
guard = torch.full((4096,), 7.0, device=DEV)      # whatever lies near `out` must stay as it is
tq.tq_attend_decode(groups, heads, T, qpk, Q, 1.0 / math.sqrt(HD), out, ws)
tq.tq_plan_status(gK[0].plan)
good = out.clone()
assert bool(torch.isfinite(good).all()) and float(good.abs().sum()) > 0
bad = dict(groups[1])
bad["v_channels"] = groups[1]["v_channels"].clone()
bad["v_channels"][1, 5] = HD + 1000                # outside the output row: the debug build must not store through it
out2 = torch.zeros_like(out)
tq.tq_attend_decode([groups[0], bad], heads, T, qpk, Q, 1.0 / math.sqrt(HD), out2, ws)
try:
    tq.tq_plan_status(gK[0].plan)
    raise SystemExit("the bad channel index went unnoticed")
except tq.TqError as e:
    assert e.code == 8, e      # TQ_ERR_BOUNDS
col = int(groups[1]["v_channels"][1, 5])
mask = torch.ones_like(out2, dtype=torch.bool)
mask[qpk:2 * qpk, col] = False                      # the column that lost its value in the rows of head 1
assert torch.equal(out2[mask], good[mask]) and not bool(out2[qpk:2 * qpk, col].any())
assert bool((guard == 7.0).all())
tq.tq_plan_status(gK[0].plan)                       # the status word was cleared by the report
print("debug build ok")
"""


def test_debug_build_checks_indices_on_the_device():
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    sys.path.insert(0, root)
    from paper_2504_19874_b200 import build as tq_build
    tq_build.build(debug=True)          # a no-op when libtq_debug.so is up to date
    env = dict(os.environ, TQ_LIB_VARIANT="debug")
    r = subprocess.run([sys.executable, "-c", _CHILD, root], env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0 and "debug build ok" in r.stdout, r.stdout[-3000:] + r.stderr[-3000:]
