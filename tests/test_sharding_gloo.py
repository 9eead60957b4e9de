"""The sharded-search plumbing on CPU: two gloo ranks, each scoring its shard with the oracle, gather
their local best lists and merge; the result must equal the oracle's top-k over the whole set."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import turboquant_oracle as orc
from paper_2504_19874_b200 import sharding


def test_shard_bounds_cover_the_range_once():
    for n, world in [(10, 3), (7, 7), (5, 8), (1_000_000, 8), (0, 2)]:
        spans = [sharding.shard_bounds(n, r, world) for r in range(world)]
        assert spans[0][0] == 0 and sum(c for _, c in spans) == n
        for (s0, c0), (s1, _) in zip(spans, spans[1:]):
            assert s0 + c0 == s1
        assert max(c for _, c in spans) - min(c for _, c in spans) <= 1


def _problem():
    d, n, nq, k = 16, 501, 3, 20
    rng = np.random.default_rng(5)
    X = rng.standard_normal((n, d))
    X[100] = X[400]                      # equal vectors in different shards: equal scores, tie by id
    X[7] = X[8]
    Q = rng.standard_normal((nq, d))
    Pi, S = orc.rotation(d, 3), orc.projection(d, 4)
    c = orc.codebook(d, 2)
    idx, z, gamma, nu = orc.quant_prod(X, Pi, S, c)
    scores = orc.score(Q, orc.dequant_prod(idx, z, gamma, nu, Pi, S, c))
    return scores.astype(np.float32).astype(np.float64), k      # the exchanged scores are float32


def _rank_main(rank, world, port, out_path):
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    scores, k = _problem()
    start, count = sharding.shard_bounds(scores.shape[1], rank, world)
    vals, ids = orc.topk(scores[:, start:start + count], k)              # this rank's local search
    cs, ci = sharding.gather_candidates(torch.from_numpy(vals).float(), torch.from_numpy(ids).int(), start)
    assert cs.shape == (scores.shape[0], world * k) and ci.dtype == torch.int32
    # merge: candidates ordered by global id, so that the oracle's "lower position wins a tie" is "lower id wins"
    order = torch.argsort(ci.long(), dim=1)
    cs, ci = torch.gather(cs, 1, order), torch.gather(ci, 1, order)
    _, mpos = orc.topk(cs.double().numpy(), k)
    merged_ids = np.take_along_axis(ci.numpy(), mpos, axis=1)
    if rank == 0:
        np.save(out_path, merged_ids)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_merge_to_the_global_topk(tmp_path):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    out = str(tmp_path / "merged.npy")
    mp.spawn(_rank_main, args=(2, port, out), nprocs=2, join=True)
    scores, k = _problem()
    _, want = orc.topk(scores, k)
    assert np.array_equal(np.load(out), want)
