"""GPU parity tests (forward side): every step of the layer through the C ABI
against the CPU oracle on the same seeded inputs.  Integer results bit-exact;
floating point within the stated tolerances."""
import numpy as np
import pytest
import torch

from oracle import pquant_oracle as O
from paper_2602_22592_b200 import binding as pqb
from paper_2602_22592_b200 import inputs as I
from paper_2602_22592_b200.layer import PQLinear

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2     # max relative error of bf16 outputs / gradients
TOL_SCALE = 1e-5    # fp32-accumulated scales
TOL_RMS = 5e-3      # error of a whole tensor relative to its size (Frobenius norms)
STRICT = 1e-2       # floor of the element-wise error, as a fraction of rms(b), for results free of bf16 intermediates


def rel_err(a, b, floor=1.0):
    """max |a-b| / max(|b|, floor * rms(b)): error relative to the element or, near zero crossings, to a
    fraction of the tensor's scale.  floor = 1: results that pass through bf16 intermediates (H, q/gamma,
    dH, the scaled sign matrix), whose rounding is an ABSOLUTE error of about 2^-9 of the tensor's scale in
    every element, however small the element.  floor = STRICT (1e-2): results that do not -- the pure 1-bit
    output (exact int32 sums times fp32 scales), dB, dalpha, dX of layers without routing."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    lo = floor * np.sqrt(np.mean(b * b)) + 1e-30
    return float(np.max(np.abs(a - b) / np.maximum(np.abs(b), lo)))


def rms_err(a, b):
    """||a-b|| / ||b|| over the whole tensor.  The element-wise maximum with its rms floor lets a missing term of a
    few percent of the tensor's scale through; this does not: bf16 rounding leaves 1e-3..4e-3 here, a dropped
    contribution (the router's share of dX is 1..15 % in these cases) shows as its full share."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return float(np.sqrt(np.sum((a - b) ** 2)) / (np.sqrt(np.sum(b * b)) + 1e-30))


def f32(t):
    return t.detach().float().cpu().numpy()


def check_status():
    code, where = pqb.pq_device_status()
    assert code == 0, f"device wait timed out (where={where})"


# ------------------------------------------------------------------ pack (Eq. 3, 4, 6)
@pytest.mark.parametrize("N,K", [(32, 32), (96, 256), (512, 512), (1000 // 8 * 8, 2048), (2048, 5632)])
def test_pack_weights_bit_exact(N, K):
    N = (N + 31) // 32 * 32
    c = I.make_linear_case(1, K, N, 0, 0, seed=100 + N, with_grad=False)
    L = PQLinear(128, K, N, training=False)
    L.W = torch.from_numpy(c["W"]).cuda()
    L.pack()
    torch.cuda.synchronize()
    mu, lam = O.weight_scales(c["W"])
    S = O.binarize(c["W"], mu)
    sc = f32(L.w_scales)
    assert abs(sc[0] - lam) <= TOL_SCALE * abs(lam) and abs(sc[1] - mu) <= TOL_SCALE * abs(lam)
    assert sc[1] == mu and sc[0] == lam          # in practice bit-identical
    assert np.array_equal(L.w_s8.cpu().numpy(), S)
    assert np.array_equal(L.w_bits.cpu().numpy().view(np.uint32), O.pack_bits(S))


def test_pack_constant_matrix_and_ties():
    W = np.full((64, 64), 0.125, np.float32)
    L = PQLinear(128, 64, 64, training=False)
    L.W = torch.from_numpy(W).cuda()
    L.pack()
    assert np.all(L.w_s8.cpu().numpy() == 1)      # Sign(0) := +1
    assert np.all(L.w_bits.cpu().numpy().view(np.uint32) == 0xFFFFFFFF)


# ------------------------------------------------------------------ tensor-core engine, raw accumulators
@pytest.mark.parametrize("M,N,K", [(128, 256, 128), (256, 512, 512), (392, 520, 1040), (8, 16, 16)])
def test_engine_int8_accumulators_bit_exact(M, N, K):
    rng = np.random.default_rng(M + N + K)
    A = rng.integers(-128, 128, (M, K)).astype(np.int8)
    B = rng.choice([-1, 1], (N, K)).astype(np.int8)
    D = torch.full((M, N), 0x7FFFFFFF, dtype=torch.int32, device="cuda")
    pqb.pq_debug_gemm(0, M, N, K, torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), D)
    torch.cuda.synchronize()
    check_status()
    assert np.array_equal(D.cpu().numpy().astype(np.int64), O.onebit_gemm(A, B))


@pytest.mark.parametrize("tile_n", [32, 64, 128, 160, 256])
@pytest.mark.parametrize("M,N,K", [(392, 520, 1040), (2048, 4096, 256), (128, 2400, 128)])
def test_engine_int8_tile_widths_bit_exact(tile_n, M, N, K):
    # narrow tiles, the 160-wide forward tile, and shapes whose last wave is cut into pieces
    rng = np.random.default_rng(tile_n + M + N + K)
    A = rng.integers(-128, 128, (M, K)).astype(np.int8)
    B = rng.choice([-1, 1], (N, K)).astype(np.int8)
    D = torch.full((M, N), 0x7FFFFFFF, dtype=torch.int32, device="cuda")
    pqb.pq_debug_gemm_tile(0, M, N, K, torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), D, tile_n)
    torch.cuda.synchronize()
    check_status()
    assert np.array_equal(D.cpu().numpy().astype(np.int64), O.onebit_gemm(A, B))


@pytest.mark.parametrize("mode,tile_n", [(1, 96), (2, 64), (2, 128), (3, 64), (3, 192)])
def test_engine_bf16_tile_widths(mode, tile_n):
    M, N, K = 392, 1096, 520
    rng = np.random.default_rng(mode * 1000 + tile_n)
    A = I.bf16_values(rng.standard_normal((M, K)).astype(np.float32))
    B = I.bf16_values(rng.standard_normal((N, K)).astype(np.float32))
    ref = A.astype(np.float64) @ B.astype(np.float64).T
    At = torch.from_numpy(A if mode != 3 else np.ascontiguousarray(A.T)).cuda().to(torch.bfloat16)
    Bt = torch.from_numpy(B if mode == 1 else np.ascontiguousarray(B.T)).cuda().to(torch.bfloat16)
    D = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    pqb.pq_debug_gemm_tile(mode, M, N, K, At, Bt, D, tile_n)
    torch.cuda.synchronize()
    check_status()
    got = D.cpu().numpy()
    assert np.all(np.isfinite(got))
    assert np.max(np.abs(got - ref)) <= 1e-4 * np.sqrt(K) * 4


@pytest.mark.parametrize("mode", [1, 2, 3])
@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (256, 512, 512), (392, 520, 1000), (8, 16, 16)])
def test_engine_bf16_operand_forms(mode, M, N, K):
    rng = np.random.default_rng(mode * 1000 + M + N + K)
    A = I.bf16_values(rng.standard_normal((M, K)).astype(np.float32))
    B = I.bf16_values(rng.standard_normal((N, K)).astype(np.float32))
    ref = A.astype(np.float64) @ B.astype(np.float64).T
    At = torch.from_numpy(A if mode != 3 else np.ascontiguousarray(A.T)).cuda().to(torch.bfloat16)
    Bt = torch.from_numpy(B if mode == 1 else np.ascontiguousarray(B.T)).cuda().to(torch.bfloat16)
    D = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    pqb.pq_debug_gemm(mode, M, N, K, At, Bt, D)
    torch.cuda.synchronize()
    check_status()
    got = D.cpu().numpy()
    assert np.all(np.isfinite(got))
    assert np.max(np.abs(got - ref)) <= 1e-4 * np.sqrt(K) * 4


# ------------------------------------------------------------------ forward of the layer
def run_forward(c, scale_vector):
    L = PQLinear(c["T"], c["K"], c["N"], c["r"], c["E"], scale_vector=scale_vector).load_case(c)
    L.pack()
    L.forward()
    torch.cuda.synchronize()
    check_status()
    return L


def check_forward(c, L, f):
    sv = L.saved_view()
    T, E = c["T"], max(c["E"], 1)
    perm = sv["perm"].cpu().numpy()
    if c["r"] > 0 and c["E"] > 1:
        # router: indices, permutation, offsets are integers -> exact
        assert np.array_equal(sv["expert"].cpu().numpy(), f["idx"])
        assert np.array_equal(perm, f["perm"])
        assert np.array_equal(sv["offsets"].cpu().numpy(), f["offsets"])
        assert np.array_equal(sv["pos"].cpu().numpy()[perm], np.arange(T))
        assert rel_err(f32(sv["gate"]), f["gate"][perm]) <= 1e-5
        assert np.max(np.abs(f32(sv["probs"]) - f["probs"][perm])) <= 1e-6
    else:
        assert np.array_equal(perm, np.arange(T))
    # Eq. 7-9: int8 codes and gamma bit-exact
    assert np.array_equal(sv["q"].cpu().numpy(), f["q"][perm])
    assert np.array_equal(f32(sv["gamma"]), f["gamma"][perm])
    if c["r"] > 0:
        # item table covers every sorted row exactly once, one expert per item
        n_items = int(sv["n_items"].cpu()[0])
        items = sv["items"].cpu().numpy()[:n_items]
        cover = np.zeros(T, int)
        srt_e = f["idx"][perm] if c["E"] > 1 else np.zeros(T, int)
        h = f32(sv["h"]).astype(np.float64).sum(axis=0)          # hi + lo planes
        for i, (tile, e, lo, hi) in enumerate(items):
            rows = np.arange(tile * 128 + lo, tile * 128 + hi)
            cover[rows] += 1
            assert np.all(srt_e[rows] == e)
            blk = h[i * 128:(i + 1) * 128]
            assert rel_err(blk[lo:hi], f["h"][perm[rows]]) <= 1e-4
            assert np.all(blk[:lo] == 0) and np.all(blk[hi:] == 0)
        assert np.all(cover == 1)
    assert rel_err(f32(L.Y), f["Y"]) <= TOL_BF16
    assert rms_err(f32(L.Y), f["Y"]) <= TOL_RMS
    if c["r"] == 0:
        # exact int32 sums times fp32 factors, rounded once: nothing to forgive near zero crossings
        assert rel_err(f32(L.Y), f["Y"], STRICT) <= TOL_BF16


CASES = {
    "cfg1": dict(T=256, K=512, N=512, r=32, E=1, scale_vector=True, alpha=1.0, beta=1.0),
    "pure_1bit": dict(T=200, K=256, N=320, r=0, E=0),
    "dense_hp_ragged": dict(T=333, K=384, N=544, r=64, E=1),
    "routed8": dict(T=1000, K=512, N=768, r=128, E=8),
    "routed4_small_r": dict(T=520, K=256, N=256, r=16, E=4, scale_vector=True, alpha=1.5, beta=0.4),
    "routed12": dict(T=300, K=320, N=256, r=16, E=12),   # more than 8 experts: the router's 16-wide instance
    # long rows: the activation quantiser keeps a row in registers of 1, 2 or 4 warps, or re-reads it
    "k2048": dict(T=70, K=2048, N=64, r=0, E=0),
    "k4096_routed": dict(T=200, K=4096, N=64, r=16, E=4),
    "k5632": dict(T=130, K=5632, N=96, r=0, E=0),
    "k8704": dict(T=40, K=8704, N=64, r=0, E=0),
}


@pytest.mark.parametrize("name", list(CASES))
def test_forward_matches_oracle(name):
    kw = dict(CASES[name])
    sv = kw.pop("scale_vector", False)
    c = I.make_linear_case(kw.pop("T"), kw.pop("K"), kw.pop("N"), kw.pop("r"), kw.pop("E"), seed=7, scale_vector=sv, **kw)
    f = O.linear_forward(c["X"], c["W"], c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    L = run_forward(c, sv)
    check_forward(c, L, f)


@pytest.mark.parametrize("E,zero", [(1, "A"), (1, "B"), (8, "B"), (4, "alpha")])
def test_forward_with_hp_branch_zeroed_is_the_pure_onebit_layer(E, zero):
    # Eq. 11 with the HP term at zero: the kernels still run both accumulators, and what is left is the 1-bit
    # branch alone -- exact integers times fp32 scales -- so the output must meet the tolerance element by element
    # with the strict floor, and equal the oracle's pure 1-bit layer.
    c = I.make_linear_case(450, 512, 544, 64, E, seed=13)
    if zero == "alpha":
        c["alpha"][:] = 0.0
    else:
        c[zero] = np.zeros_like(c[zero])
    f = O.linear_forward(c["X"], c["W"], c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    pure = O.linear_forward(c["X"], c["W"], beta=c["beta"])
    assert np.array_equal(f["Y"], pure["Y"])
    L = run_forward(c, False)
    assert rel_err(f32(L.Y), pure["Y"], STRICT) <= TOL_BF16
    assert rms_err(f32(L.Y), pure["Y"]) <= 1e-3


def test_forward_degenerate_rows_and_experts():
    # an all-zero token, a constant-sign row, and a router that sends every token to one expert
    c = I.make_linear_case(300, 256, 256, 32, 4, seed=9, zipf=False)
    c["X"][7] = 0.0
    c["Wr"][:] = 0.0
    c["Wr"][2] = I.bf16_values(np.full(256, 0.5, np.float32))
    c["X"] = I.bf16_values(np.abs(c["X"]))        # positive activations -> expert 2 wins everywhere except the zero row
    f = O.linear_forward(c["X"], c["W"], c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    assert f["idx"][7] == 0 and np.all(np.delete(f["idx"], 7) == 2)
    L = run_forward(c, False)
    check_forward(c, L, f)


def test_forward_is_deterministic():
    c = I.make_linear_case(512, 512, 512, 64, 4, seed=3)
    L = run_forward(c, False)
    y1 = L.Y.clone()
    L.forward()
    torch.cuda.synchronize()
    assert torch.equal(y1, L.Y)


def test_argument_errors_are_reported():
    d = pqb.make_desc(128, 100, 64)               # K not a multiple of 32
    assert pqb.pq_saved_bytes(d) == 0
    L = PQLinear(128, 64, 64, 32, 1)
    with pytest.raises(pqb.PqError) as ei:
        pqb.pq_linear_forward(L.desc, None, L.w_bits, L.w_s8, L.w_scales, None, None, None, None, None, L.Y, L.saved, L.ws_fwd)
    assert ei.value.status == pqb.PQ_ERR_NULL
    small = torch.empty(16, dtype=torch.uint8, device="cuda")
    c = I.make_linear_case(128, 64, 64, 32, 1, seed=1)
    L.load_case(c)
    with pytest.raises(pqb.PqError) as ei:
        pqb.pq_linear_forward(L.desc, L.X, L.w_bits, L.w_s8, L.w_scales, L.A, L.B, None, L.alpha, L.beta, L.Y, L.saved, small)
    assert ei.value.status == pqb.PQ_ERR_WORKSPACE


# ------------------------------------------------------------------ INT8 high-precision branch: expert quantisation (Sec. 3.2)
@pytest.mark.parametrize("E,r,K,N", [(1, 32, 512, 512), (8, 128, 2048, 1024), (3, 40, 2080, 992), (8, 160, 3200, 8640)])
def test_pack_experts_bit_exact(E, r, K, N):
    c = I.make_linear_case(8, K, N, r, E, seed=17, exact_quota=False, with_grad=False)
    d = pqb.make_desc(8, K, N, r, E)
    A = torch.from_numpy(c["A"]).cuda().to(torch.bfloat16)
    B = torch.from_numpy(c["B"]).cuda().to(torch.bfloat16)
    A8 = torch.zeros((E, r, K), dtype=torch.int8, device="cuda")
    B8 = torch.zeros((E, N, r), dtype=torch.int8, device="cuda")
    sc = torch.zeros((E, 2), dtype=torch.float32, device="cuda")
    ws = torch.empty(pqb.pq_workspace_bytes(d, pqb.PQ_PHASE_PACK), dtype=torch.uint8, device="cuda")
    for _ in range(2):          # twice in a row: the scratch of the first call must not leak into the second
        pqb.pq_pack_experts(d, A, B, A8, B8, sc, ws)
    torch.cuda.synchronize()
    wA8, gA, wB8, gB = O.quantize_experts(c["A"], c["B"])
    assert np.array_equal(sc.cpu().numpy()[:, 0], gA) and np.array_equal(sc.cpu().numpy()[:, 1], gB)
    assert np.array_equal(A8.cpu().numpy(), wA8) and np.array_equal(B8.cpu().numpy(), wB8)


HP8_CASES = {
    "dense_r32": dict(T=333, K=384, N=544, r=32, E=1),
    "routed8_r128": dict(T=1000, K=512, N=768, r=128, E=8),
    "routed4_r16_vec": dict(T=520, K=256, N=256, r=16, E=4, scale_vector=True, alpha=1.5, beta=0.4),
    "routed3_r48_long_rows": dict(T=200, K=4096, N=96, r=48, E=3),
}


@pytest.mark.parametrize("name", list(HP8_CASES))
def test_forward_int8_hp_branch_matches_oracle(name):
    # Sec. 3.2: the HP branch at 8-bit precision on the int8 activation codes.  Integers (codes of h and their scale,
    # hence the exact int32 sums behind them) bit for bit; Y within the bf16 tolerance of the oracle's INT8 forward.
    kw = dict(HP8_CASES[name])
    sv = kw.pop("scale_vector", False)
    c = I.make_linear_case(kw.pop("T"), kw.pop("K"), kw.pop("N"), kw.pop("r"), kw.pop("E"), seed=19, scale_vector=sv, **kw)
    if sv:
        c["alpha"] = (c["alpha"] * np.linspace(0.8, 1.2, c["N"])).astype(np.float32)
        c["beta"] = (c["beta"] * np.linspace(1.2, 0.8, c["N"])).astype(np.float32)
    f = O.linear_forward(c["X"], c["W"], c["A"], c["B"], c["Wr"], c["alpha"], c["beta"], hp_int8=True)
    L = PQLinear(c["T"], c["K"], c["N"], c["r"], c["E"], scale_vector=sv, guard=True).load_case(c)
    L.pack()
    L.pack_experts()
    L.forward_hp8()
    torch.cuda.synchronize()
    check_status()
    assert L.check_guards() == 0
    assert np.array_equal(L.A8.cpu().numpy(), f["A8"]) and np.array_equal(L.B8.cpu().numpy(), f["B8"])
    svw = L.saved_view()
    perm = svw["perm"].cpu().numpy()
    assert np.array_equal(svw["q"].cpu().numpy(), f["q"][perm])
    if c["E"] > 1:
        assert np.array_equal(svw["expert"].cpu().numpy(), f["idx"])
    h8 = L.hp8_view()
    qh, gh = h8["qh"].cpu().numpy(), h8["gamma_h"].cpu().numpy()
    items = svw["items"].cpu().numpy()[:int(svw["n_items"].cpu()[0])]
    seen = 0
    for i, (tile, e, lo, hi) in enumerate(items):
        rows = np.arange(tile * 128 + lo, tile * 128 + hi)
        tokens = perm[rows]
        assert np.array_equal(qh[i * 128 + lo:i * 128 + hi], f["qh"][tokens])         # codes of h: exact int32 sums behind them
        assert np.array_equal(gh[i * 128 + lo:i * 128 + hi], f["gamma_h"][tokens])
        assert not np.any(qh[i * 128:i * 128 + lo]) and not np.any(qh[i * 128 + hi:(i + 1) * 128])
        seen += len(rows)
    assert seen == c["T"]
    assert rel_err(f32(L.Y), f["Y"]) <= TOL_BF16
    assert rms_err(f32(L.Y), f["Y"]) <= TOL_RMS
    # and it is the INT8 branch, not the bf16 one
    fb = O.linear_forward(c["X"], c["W"], c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    assert rms_err(f["Y"], fb["Y"]) > 2e-3


def test_forward_int8_hp_rejects_odd_width():
    L = PQLinear(128, 64, 64, 40, 1)
    c = I.make_linear_case(128, 64, 64, 40, 1, seed=1)
    L.load_case(c)
    L.pack()
    L.pack_experts()
    with pytest.raises(pqb.PqError) as ei:
        L.forward_hp8()
    assert ei.value.status == pqb.PQ_ERR_SHAPE


@pytest.mark.parametrize("T,K,N,r,E", [(300, 384, 544, 32, 4), (129, 256, 320, 16, 8), (64, 512, 96, 64, 2)])
def test_all_experts_with_unit_gates_is_the_dense_layer_of_width_E_r(T, K, N, r, E):
    # Sec. 3.3, the special case in which routing reduces to a dense branch: top_k = E with unit gates.  The oracle's
    # sum over all experts (weights one) is the expected value; the same call on a dense layer built from the stacked A
    # and the side-by-side B must give the same bits (it is the same arithmetic).
    c = I.make_linear_case(T, K, N, r, E, seed=31)
    L = PQLinear(T, K, N, r, E, guard=True).load_case(c)      # buffers and packed weights; its own desc is top-1
    L.pack()
    d = pqb.make_desc(T, K, N, r, E, top_k=E, unit_gates=True)
    saved = torch.empty(pqb.pq_saved_bytes(d), dtype=torch.uint8, device="cuda")
    ws = torch.empty(pqb.pq_workspace_bytes(d, pqb.PQ_PHASE_FWD), dtype=torch.uint8, device="cuda")
    assert saved.numel() > 0 and ws.numel() > 0
    Y = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
    pqb.pq_linear_forward(d, L.X, L.w_bits, L.w_s8, L.w_scales, L.A, L.B, None, L.alpha, L.beta, Y, saved, ws)
    torch.cuda.synchronize()
    check_status()
    assert L.check_guards() == 0
    f1 = O.linear_forward(c["X"], c["W"], alpha=c["alpha"], beta=c["beta"])                 # the 1-bit branch alone
    z = O.hp_branch_all_experts(c["X"], c["A"], c["B"], np.ones((T, E)))
    al = np.broadcast_to(np.asarray(c["alpha"], dtype=np.float64).reshape(-1), (N,))
    want = O.round_to_bf16(al[None, :] * z + f1["Y64"])
    assert rel_err(f32(Y), want) <= TOL_BF16 and rms_err(f32(Y), want) <= TOL_RMS
    # the dense layer of width E r
    Ld = PQLinear(T, K, N, r * E, 1).load_case(c)
    Ld.A = L.A.reshape(1, E * r, K).contiguous()
    Ld.B = L.B.permute(1, 0, 2).reshape(1, N, E * r).contiguous()
    Ld.Wr = None
    Ld.pack()
    Ld.forward()
    torch.cuda.synchronize()
    assert torch.equal(Ld.Y, Y)
    # not what top-1 routing gives
    L.forward()
    torch.cuda.synchronize()
    assert not torch.equal(L.Y, Y)


def test_all_experts_mode_limits():
    d = pqb.make_desc(64, 256, 256, 32, 4, top_k=4)                       # without the unit-gate flag
    assert pqb.pq_saved_bytes(d) == 0 and pqb.pq_workspace_bytes(d, pqb.PQ_PHASE_FWD) == 0
    d = pqb.make_desc(64, 256, 256, 64, 4, top_k=4, unit_gates=True)      # E r > 128
    assert pqb.pq_saved_bytes(d) == 0
    d = pqb.make_desc(64, 256, 256, 32, 4, top_k=2, unit_gates=True)      # neither 1 nor E
    assert pqb.pq_saved_bytes(d) == 0
    d = pqb.make_desc(64, 256, 256, 32, 4, top_k=4, unit_gates=True)
    assert pqb.pq_workspace_bytes(d, pqb.PQ_PHASE_BWD) == 0               # forward only
