"""GPU tests of the library's safety nets: a bounded device-side wait that really runs out (and the library
carrying on afterwards), and canary bands around every buffer the kernels write."""
import numpy as np
import pytest
import torch

from oracle import pquant_oracle as O
from paper_2602_22592_b200 import binding as pqb
from paper_2602_22592_b200 import inputs as I
from paper_2602_22592_b200.layer import GUARD_BYTES, PQLinear
from test_gpu_forward import check_status

pytestmark = pytest.mark.gpu


def test_bounded_wait_runs_out_and_the_next_call_is_correct():
    # Nothing is broken here: the spin limit is cut to one clock cycle for ONE launch of the engine's test
    # GEMM, so the first wait that does not succeed at once (operands still on their way, or the long wait of
    # the epilogue warps for a whole contraction) gives up.  The kernel must come back, report
    # PQ_ERR_TIMEOUT through the status word, and leave the context usable.
    M, N, K = 1024, 2048, 16384
    rng = np.random.default_rng(1)
    A = torch.from_numpy(rng.integers(-128, 128, (M, K)).astype(np.int8)).cuda()
    B = torch.from_numpy(rng.choice([-1, 1], (N, K)).astype(np.int8)).cuda()
    D = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    check_status()
    pqb.pq_set_option(pqb.PQ_OPT_SPIN_CYCLES, 1)
    try:
        pqb.pq_debug_gemm(0, M, N, K, A, B, D)
        code, where = pqb.pq_device_status()
    finally:
        pqb.pq_set_option(pqb.PQ_OPT_SPIN_CYCLES, 0)      # back to the default of about two seconds
    assert code == pqb.PQ_ERR_TIMEOUT
    assert where in (1, 2, 3)                               # producer, MMA issuer or epilogue
    assert pqb.pq_device_status() == (0, 0)                 # reading the status clears it
    # the next call, with the normal limit, is exact again
    pqb.pq_debug_gemm(0, M, N, K, A, B, D)
    torch.cuda.synchronize()
    check_status()
    rows = rng.choice(M, 24, replace=False)
    want = A[rows].cpu().numpy().astype(np.int64) @ B.cpu().numpy().astype(np.int64).T
    assert np.array_equal(D[rows].cpu().numpy().astype(np.int64), want)

def test_grid_barrier_of_the_streaming_decode_kernel_runs_out_and_recovers():
    # The streaming decode kernel's CTAs meet at one grid barrier with a bounded wait.  With a limit of one cycle the first
    # poll that finds a CTA still missing gives up: that CTA records PQ_ERR_TIMEOUT and skips the rest of its work (nothing
    # after the barrier reads what a missing CTA would have written), every CTA still leaves the barrier words balanced,
    # and the next call with the normal limit is exact.  Only this kernel runs under the short limit.
    c = I.make_linear_case(4, 512, 2048, 32, 4, seed=53)
    L = PQLinear(4, 512, 2048, 32, 4, training=False, dump_acc=True).load_case(c)
    pqb.pq_set_option(pqb.PQ_OPT_DECODE_STREAM, 2)
    try:
        L.pack(bits_only=True)
        if L.w_bits_il is None:
            L.pack_decode()
        L.decode()
        torch.cuda.synchronize()
        check_status()
        want = L.Y.clone()
        acc = L.decode_view()["acc"].clone()
        pqb.pq_set_option(pqb.PQ_OPT_SPIN_CYCLES, 1)
        try:
            L.decode()
            code, where = pqb.pq_device_status()
        finally:
            pqb.pq_set_option(pqb.PQ_OPT_SPIN_CYCLES, 0)
        assert code == pqb.PQ_ERR_TIMEOUT and where == 4
        assert pqb.pq_device_status() == (0, 0)
        for _ in range(2):
            L.Y.zero_()
            L.decode()
            torch.cuda.synchronize()
            check_status()
            assert torch.equal(L.Y, want) and torch.equal(L.decode_view()["acc"], acc)
    finally:
        pqb.pq_set_option(pqb.PQ_OPT_DECODE_STREAM, 1)


@pytest.mark.parametrize("shape", [dict(T=333, K=384, N=544, r=64, E=1), dict(T=1000, K=512, N=768, r=128, E=8),
                                   dict(T=200, K=256, N=320, r=0, E=0), dict(T=130, K=5632, N=96, r=16, E=4)])
def test_training_kernels_stay_inside_their_buffers(shape):
    c = I.make_linear_case(shape["T"], shape["K"], shape["N"], shape["r"], shape["E"], seed=51)
    L = PQLinear(c["T"], c["K"], c["N"], c["r"], c["E"], guard=True).load_case(c)
    assert L.check_guards() == 0
    L.pack()
    L.forward()
    L.backward()
    torch.cuda.synchronize()
    check_status()
    assert L.check_guards() == 0
    # ... and the guarded run still computes the layer
    f = O.linear_forward(c["X"], c["W"], c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    perm = L.saved_view()["perm"].cpu().numpy()
    assert np.array_equal(L.saved_view()["q"].cpu().numpy(), f["q"][perm])


@pytest.mark.parametrize("shape", [dict(T=5, K=2080, N=992, r=40, E=3), dict(T=16, K=512, N=2048, r=64, E=8),
                                   dict(T=3, K=1024, N=64, r=0, E=0)])
def test_decode_kernels_stay_inside_their_buffers(shape):
    c = I.make_linear_case(shape["T"], shape["K"], shape["N"], shape["r"], shape["E"], seed=52, exact_quota=False, with_grad=False)
    L = PQLinear(c["T"], c["K"], c["N"], c["r"], c["E"], training=False, dump_acc=True, guard=True).load_case(c)
    L.pack(bits_only=True)
    L.decode()
    torch.cuda.synchronize()
    check_status()
    assert L.check_guards() == 0
    mu, lam = O.weight_scales(c["W"])
    f = O.decode_forward(c["X"], O.pack_bits(O.binarize(c["W"], mu)), lam, c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    assert np.array_equal(L.decode_view()["acc"].cpu().numpy().astype(np.int64), f["acc"])


def test_guard_check_sees_a_stray_byte():
    # the checker itself: one byte written just past a buffer (by torch, from the host side) is counted
    L = PQLinear(128, 64, 64, guard=True)
    assert L.check_guards() == 0
    raw, nbytes = L._guards[0]
    raw[GUARD_BYTES + nbytes] = 0
    raw[GUARD_BYTES - 1] = 1
    assert L.check_guards() == 2
