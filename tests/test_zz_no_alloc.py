"""pq_pack_weights_static: the weight pack for callers that cannot allocate device
memory (their memory was handed out once by someone else, or an allocation's
implicit synchronisation is not acceptable where they run).  Its reduction
scratch is a fixed array inside the library, so the test checks two things a
shared, never-cleared buffer could get wrong: the result matches the regular
entry point, and a second call on different data is not polluted by the first.

Collected last on purpose: a failure here cannot hide the other tests' results
in a run that stops at the first failure."""
import numpy as np
import pytest
import torch

from oracle import pquant_oracle as O
from paper_2602_22592_b200 import binding as pqb
from paper_2602_22592_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _pack_both(W):
    N, K = W.shape
    d = pqb.make_desc(128, K, N)
    Wd = torch.from_numpy(W).cuda()
    out = []
    for static in (False, True):
        bits = torch.zeros((N, K // 32), dtype=torch.int32, device="cuda")
        s8 = torch.zeros((N, K), dtype=torch.int8, device="cuda")
        scales = torch.zeros(2, dtype=torch.float32, device="cuda")
        if static:
            pqb.pq_pack_weights_static(d, Wd, bits, s8, scales)
        else:
            ws = torch.empty(pqb.pq_workspace_bytes(d, pqb.PQ_PHASE_PACK), dtype=torch.uint8, device="cuda")
            pqb.pq_pack_weights(d, Wd, bits, s8, scales, ws)
        torch.cuda.synchronize()
        out.append((bits.cpu().numpy(), s8.cpu().numpy(), scales.cpu().numpy()))
    return out


def test_static_pack_matches_regular_pack_twice_in_a_row():
    # two calls in a row, the second on a smaller matrix with a very different mean:
    # stale partial sums of the first call left in the shared scratch must not leak in
    first = I.make_linear_case(1, 2048, 1536, 0, 0, seed=71, with_grad=False)["W"]
    second = (I.make_linear_case(1, 512, 320, 0, 0, seed=72, with_grad=False)["W"] + np.float32(0.01)).astype(np.float32)
    for W in (first, second):
        (bits_r, s8_r, sc_r), (bits_s, s8_s, sc_s) = _pack_both(W)
        assert np.all(np.abs(sc_s - sc_r) <= 1e-5 * np.abs(sc_r[0]))      # lam, mu: fp32-accumulated-scale tolerance
        assert np.array_equal(bits_s, bits_r)
        assert np.array_equal(s8_s, s8_r)


def test_static_pack_back_to_back_without_a_sync_matches_the_oracle():
    # The documented way to share the one scratch array: several calls in stream order, nothing in between.  A large
    # matrix, a small one with a shifted mean, a large one again: every call must see its own partial sums, not its
    # neighbour's, and each result is checked against the CPU oracle (Eq. 3, 4, 6), bit for bit.
    mats = [I.make_linear_case(1, 2048, 1536, 0, 0, seed=73, with_grad=False)["W"],
            (I.make_linear_case(1, 256, 96, 0, 0, seed=74, with_grad=False)["W"] - np.float32(0.015)).astype(np.float32),
            (I.make_linear_case(1, 1024, 2048, 0, 0, seed=75, with_grad=False)["W"] + np.float32(0.004)).astype(np.float32)]
    dev = [torch.from_numpy(W).cuda() for W in mats]
    outs = []
    for W in mats:
        N, K = W.shape
        outs.append((torch.zeros((N, K // 32), dtype=torch.int32, device="cuda"), torch.zeros((N, K), dtype=torch.int8, device="cuda"),
                     torch.zeros(2, dtype=torch.float32, device="cuda")))
    # warm up the entry point (its first call on a device looks up the array's address), then measure free memory
    pqb.pq_pack_weights_static(pqb.make_desc(128, mats[1].shape[1], mats[1].shape[0]), dev[1], *outs[1])
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for W, Wd, (bits, s8, sc) in zip(mats, dev, outs):
        pqb.pq_pack_weights_static(pqb.make_desc(128, W.shape[1], W.shape[0]), Wd, bits, s8, sc)     # no synchronisation in between
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before       # the calls took no device memory
    for W, (bits, s8, sc) in zip(mats, outs):
        mu, lam = O.weight_scales(W)
        S = O.binarize(W, mu)
        got = sc.cpu().numpy()
        assert abs(got[0] - lam) <= 1e-5 * abs(lam) and abs(got[1] - mu) <= 1e-5 * abs(lam)
        assert got[0] == lam and got[1] == mu
        assert np.array_equal(s8.cpu().numpy(), S)
        assert np.array_equal(bits.cpu().numpy().view(np.uint32), O.pack_bits(S))


def test_static_pack_rejects_oversized_and_bad_arguments():
    dummy = torch.zeros(64, dtype=torch.float32, device="cuda")
    too_big = pqb.make_desc(128, 8192, 8192 + 32)            # 67.4 M elements > 67,108,864
    with pytest.raises(pqb.PqError) as ei:
        pqb.pq_pack_weights_static(too_big, dummy, dummy, dummy, dummy)
    assert ei.value.status == pqb.PQ_ERR_TOO_LARGE
    with pytest.raises(pqb.PqError) as ei:
        pqb.pq_pack_weights_static(pqb.make_desc(128, 64, 64), None, dummy, dummy, dummy)
    assert ei.value.status == pqb.PQ_ERR_NULL
