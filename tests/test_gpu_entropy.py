"""Entropy-coded index rows (Section 3.1) through the CUDA path against the oracle's coder: identical streams bit
for bit, exact round trip, and the achieved width against the entropy of the index distribution."""
import numpy as np
import pytest
import torch

import paper_2504_19874_b200 as tq
import tq_workloads as wl
from oracle import turboquant_oracle as orc
from tests import parity as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("d,bits,mode", [(128, 2, tq.TQ_MSE), (200, 3, tq.TQ_PROD), (1536, 4, tq.TQ_MSE), (264, 4, tq.TQ_PROD),
                                          (520, 1, tq.TQ_MSE)])
def test_streams_equal_the_oracle_coder_and_round_trip(d, bits, mode):
    su = P.Setup(d, bits, mode)
    bm = su.mse_bits
    n = 257
    X = torch.randn((n, d), generator=torch.Generator().manual_seed(d + bits)).to(DEV)
    idx = su.quantize(X)[0]
    p = orc.index_probabilities(d, orc.codebook(d, bm))
    lengths = orc.huffman_lengths(p) if bm > 0 else None
    codes = orc.canonical_codes(lengths)
    packed, offsets = tq.tq_entropy_pack(su.plan, lengths, n, idx)
    tq.tq_plan_status(su.plan)
    packed_h, off_h = packed.cpu().numpy(), offsets.cpu().numpy()
    sym = orc.unpack_bits(idx.cpu().numpy(), bm, d)
    assert off_h[0] == 0 and np.all(np.diff(off_h) % 4 == 0)
    for r in (0, 1, n // 2, n - 1):
        want, nbits = orc.entropy_encode_row(sym[r], lengths, codes)
        row = packed_h[off_h[r]:off_h[r + 1]]
        assert row.size == (nbits + 31) // 32 * 4
        assert np.array_equal(row[:want.size], want) and not row[want.size:].any()
        assert np.array_equal(orc.entropy_decode_row(row, d, lengths, codes), sym[r])
    back = torch.full_like(idx, 0xEE)
    tq.tq_entropy_unpack(su.plan, lengths, n, packed, offsets, back)
    torch.cuda.synchronize()
    assert torch.equal(back, idx)


def test_library_lengths_are_an_optimal_code_too():
    for d, b in ((1536, 4), (200, 2), (64, 3)):
        c = orc.codebook(d, b).astype(np.float32)
        p = orc.index_probabilities(d, c)
        got = tq.tq_entropy_lengths(d, b, c).astype(int)
        want = orc.huffman_lengths(p).astype(int)
        assert sum(2.0 ** -l for l in got) == 1.0
        assert abs(float((p * got).sum()) - float((p * want).sum())) < 1e-9      # equal expected length (ties may be split differently)


def test_achieved_width_at_b4_against_the_entropy():
    cfg = wl.CONFIGS["c4"]
    su = P.Setup(cfg.d, 4, tq.TQ_MSE, cfg.pi_seed, cfg.s_seed)
    n = 20000
    X = wl.database(cfg, n, device=DEV)
    idx = su.quantize(X)[0]
    c = orc.codebook(cfg.d, 4)
    p = orc.index_probabilities(cfg.d, c)
    lengths = tq.tq_entropy_lengths(cfg.d, 4, c.astype(np.float32))
    packed, offsets = tq.tq_entropy_pack(su.plan, lengths, n, idx)
    bits_per_coord = packed.numel() * 8 / (n * cfg.d)
    entropy = float(-(p * np.log2(p)).sum())
    expected = float((p * lengths).sum())
    print(f"b=4: entropy {entropy:.4f}, Huffman expectation {expected:.4f}, achieved {bits_per_coord:.4f} bits per coordinate")
    assert abs(entropy - 3.8) < 0.05                       # Section 3.1
    assert abs(bits_per_coord - (expected + 16.0 / cfg.d)) < 0.004   # rows end on 32-bit words: + 16 / d bits on average
    assert bits_per_coord < 3.9
    back = torch.empty_like(idx)
    tq.tq_entropy_unpack(su.plan, lengths, n, packed, offsets, back)
    assert torch.equal(back, idx)


def test_a_buffer_that_is_too_small_is_reported():
    su = P.Setup(128, 2, tq.TQ_MSE)
    X = torch.randn((64, 128), generator=torch.Generator().manual_seed(2)).to(DEV)
    idx = su.quantize(X)[0]
    lengths = np.array([2, 2, 2, 2], dtype=np.uint8)
    packed, offsets = tq.tq_entropy_pack(su.plan, lengths, 64, idx)
    assert packed.numel() == 64 * 32
    import ctypes
    small = torch.zeros(100, dtype=torch.uint8, device=DEV)
    rc = tq.lib().tq_entropy_pack(su.plan.handle, lengths.ctypes.data_as(ctypes.c_void_p), 64, idx.data_ptr(), offsets.data_ptr(),
                                  small.data_ptr(), 100, None)
    assert rc == 0
    with pytest.raises(tq.TqError):
        tq.tq_plan_status(su.plan)
    with pytest.raises(tq.TqError):                       # lengths that no prefix code has
        tq.tq_entropy_pack(su.plan, np.array([1, 1, 1, 2], dtype=np.uint8), 64, idx)
