"""GPU parity of the FFN-level decoupling (Eq. 11, Table 1): Y = alpha FFN_INT8[:r](x) + beta FFN_INT1[r:](x) through the C
ABI against the CPU oracle.  Every integer stage bit for bit (codes of x, exact sums and hidden codes of the INT8 FFN,
and -- replayed on the hidden activation the GPU itself produced -- the codes feeding the 1-bit down projection); the
bf16 tensors within the tolerance."""
import numpy as np
import pytest
import torch

from oracle import pquant_oracle as O
from paper_2602_22592_b200 import binding as pqb
from paper_2602_22592_b200 import inputs as I
from test_gpu_forward import TOL_BF16, TOL_RMS, check_status, f32, rel_err, rms_err

pytestmark = pytest.mark.gpu


def _weights(T, Dm, F1, r, seed):
    rng = np.random.default_rng(seed)
    X = I.bf16_values(rng.standard_normal((T, Dm)).astype(np.float32))
    s = 1.0 / np.sqrt(Dm)
    Wg, Wu = (rng.standard_normal((F1, Dm)) * s).astype(np.float32), (rng.standard_normal((F1, Dm)) * s).astype(np.float32)
    Wd = (rng.standard_normal((Dm, F1)) / np.sqrt(F1)).astype(np.float32)
    G = I.bf16_values((rng.standard_normal((r, Dm)) * s).astype(np.float32))
    U = I.bf16_values((rng.standard_normal((r, Dm)) * s).astype(np.float32))
    D = I.bf16_values((rng.standard_normal((Dm, r)) / np.sqrt(r)).astype(np.float32))
    return X, Wg, Wu, Wd, G, U, D


def _pack(W):
    N, K = W.shape
    d = pqb.make_desc(128, K, N)
    Wd = torch.from_numpy(W).cuda()
    bits = torch.empty((N, K // 32), dtype=torch.int32, device="cuda")
    s8 = torch.empty((N, K), dtype=torch.int8, device="cuda")
    sc = torch.empty(2, dtype=torch.float32, device="cuda")
    ws = torch.empty(pqb.pq_workspace_bytes(d, pqb.PQ_PHASE_PACK), dtype=torch.uint8, device="cuda")
    pqb.pq_pack_weights(d, Wd, bits, s8, sc, ws)
    return s8, sc


def _pack8(A, B):
    # one "expert": A [r, K], B [N, r] -> int8 codes and {gamma_A, gamma_B}
    r, K = A.shape
    N = B.shape[0]
    d = pqb.make_desc(128, K, N, r, 1)
    At = torch.from_numpy(A).cuda().to(torch.bfloat16).view(1, r, K).contiguous()
    Bt = torch.from_numpy(B).cuda().to(torch.bfloat16).view(1, N, r).contiguous()
    A8 = torch.empty((1, r, K), dtype=torch.int8, device="cuda")
    B8 = torch.empty((1, N, r), dtype=torch.int8, device="cuda")
    sc = torch.empty((1, 2), dtype=torch.float32, device="cuda")
    ws = torch.empty(pqb.pq_workspace_bytes(d, pqb.PQ_PHASE_PACK), dtype=torch.uint8, device="cuda")
    pqb.pq_pack_experts(d, At, Bt, A8, B8, sc, ws)
    return A8, B8, sc


@pytest.mark.parametrize("T,Dm,F1,r", [(200, 256, 480, 32), (333, 512, 1312, 128), (1000, 384, 1024, 64)])
def test_ffn_decoupled_forward_matches_oracle(T, Dm, F1, r):
    X, Wg, Wu, Wd, G, U, D = _weights(T, Dm, F1, r, seed=T + r)
    alpha, beta = 2.0, 0.2
    f = O.ffn_decoupled_forward(X, Wg, Wu, Wd, G, U, D, alpha, beta)
    g_s8, g_sc = _pack(Wg)
    u_s8, u_sc = _pack(Wu)
    d_s8, d_sc = _pack(Wd)
    G8, D8, sc_gd = _pack8(G, D)
    U8, _, sc_ud = _pack8(U, D)
    hp = torch.stack([sc_gd[0, 0], sc_ud[0, 0], sc_gd[0, 1]]).contiguous()
    torch.cuda.synchronize()
    assert np.array_equal(G8.cpu().numpy()[0], f["G8"]) and np.array_equal(U8.cpu().numpy()[0], f["U8"]) and np.array_equal(D8.cpu().numpy()[0], f["D8"])
    assert np.array_equal(hp.cpu().numpy(), np.array([f["gG"], f["gU"], f["gD"]], np.float32))
    d = pqb.make_ffn_desc(T, Dm, F1, r)
    ws = torch.full((pqb.pq_ffn_workspace_bytes(d) + 8192,), 0xA5, dtype=torch.uint8, device="cuda")      # canary band behind
    Xd = torch.from_numpy(X).cuda().to(torch.bfloat16)
    Y = torch.empty((T, Dm), dtype=torch.bfloat16, device="cuda")
    al, be = torch.full((1,), alpha, device="cuda"), torch.full((1,), beta, device="cuda")
    pqb.pq_ffn_forward(d, Xd, g_s8, g_sc, u_s8, u_sc, d_s8, d_sc, G8, U8, D8, hp, al, be, Y, ws[:-8192])
    torch.cuda.synchronize()
    check_status()
    assert bool((ws[-8192:] == 0xA5).all())
    v = pqb.pq_ffn_view_init(d, ws[:-8192])
    # INT8 FFN: exact sums, hidden codes and scales
    assert np.array_equal(v["g_int"].cpu().numpy()[:T].astype(np.int64), f["hp"]["g_int"])
    assert np.array_equal(v["u_int"].cpu().numpy()[:T].astype(np.int64), f["hp"]["u_int"])
    assert np.array_equal(v["qm"].cpu().numpy()[:T], f["hp"]["qm"])
    assert np.array_equal(v["gamma_m"].cpu().numpy()[:T], f["hp"]["gamma_m"])
    # 1-bit FFN: gate and up outputs are exact integers times fp32 scales, rounded once
    assert rel_err(f32(v["G1"]), f["gate"]["Y"], 1e-2) <= TOL_BF16 and rel_err(f32(v["U1"]), f["up"]["Y"], 1e-2) <= TOL_BF16
    assert rms_err(f32(v["M1"]), f["m1"]) <= TOL_RMS and rel_err(f32(v["M1"]), f["m1"]) <= TOL_BF16
    # the down projection on the hidden activation the GPU produced: codes and scales exact
    q_m1, g_m1 = O.act_quant(f32(v["M1"]))
    assert np.array_equal(v["q_m1"].cpu().numpy(), q_m1) and np.array_equal(v["gamma_m1"].cpu().numpy(), g_m1)
    # and the sum of the two branches
    assert rel_err(f32(Y), f["Y"]) <= TOL_BF16
    assert rms_err(f32(Y), f["Y"]) <= TOL_RMS
    # both branches matter in it
    only1 = O.round_to_bf16(beta * f["down"]["y1"])
    assert rms_err(only1, f["Y"]) > 0.2


def test_ffn_rejects_bad_shapes():
    assert pqb.pq_ffn_workspace_bytes(pqb.make_ffn_desc(128, 256, 480, 24)) == 0       # r not a multiple of 16
    assert pqb.pq_ffn_workspace_bytes(pqb.make_ffn_desc(128, 250, 480, 32)) == 0
    assert pqb.pq_ffn_workspace_bytes(pqb.make_ffn_desc(128, 256, 480, 32)) > 0
