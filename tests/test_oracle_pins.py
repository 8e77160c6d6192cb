"""Pins for the CPU oracle: each check ties one oracle function to something
other than itself -- the hand-worked vectors in tests/golden, invariants the
paper's definitions force, brute force on tiny shapes, closed forms and finite
differences -- chosen so that a dropped term, a wrong sign or a transposed
operand fails at least one of them.  CPU only."""
import itertools
import os

import numpy as np
import pytest

from oracle import pquant_oracle as O
from paper_2602_22592_b200 import inputs as I

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "worked_examples.txt")


def _golden(kind):
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            parts = [p.strip() for p in line.split("|")]
            if parts[0] == kind:
                rows.append(parts[1:])
    return rows


def _mat(s):
    return np.array([[float(v) for v in row.split()] for row in s.split(";")], dtype=np.float32)


# ---------------------------------------------------------------- worked examples
@pytest.mark.parametrize("row", _golden("act_quant"))
def test_act_quant_worked(row):
    x = _mat(row[0])
    gamma = float(row[1].split()[1])
    q_exp = np.array([int(v) for v in row[2].split()[1:]])
    q, g = O.act_quant(x)
    assert g[0] == np.float32(gamma)
    assert np.array_equal(q[0], q_exp)


@pytest.mark.parametrize("row", _golden("binarize"))
def test_binarize_worked(row):
    W = _mat(row[0])
    mu_exp, lam_exp = float(row[1].split()[1]), float(row[2].split()[1])
    S_exp = _mat(row[3].split(None, 1)[1]).astype(np.int8)
    mu, lam = O.weight_scales(W)
    assert abs(float(mu) - mu_exp) <= 1e-7 and abs(float(lam) - lam_exp) <= 1e-7
    assert np.array_equal(O.binarize(W, mu), S_exp)


# ---------------------------------------------------------------- I1, I11: weights
def test_binarized_weights_two_values_and_pack_roundtrip():
    c = I.make_linear_case(8, 256, 96, 0, 0, seed=11, with_grad=False)
    mu, lam = O.weight_scales(c["W"])
    S = O.binarize(c["W"], mu)
    deq = np.float64(lam) * S
    assert set(np.unique(deq)) == {-float(lam), float(lam)}        # only +-lam
    bits = O.pack_bits(S)
    assert bits.dtype == np.uint32 and bits.nbytes * 16 == S.size * 2  # 1/16 of fp16 (App. A)
    assert np.array_equal(O.unpack_bits(bits, 256), S)
    # byte stream view: 8 weights per uint8, LSB first
    by = bits.view(np.uint8).reshape(96, 32)
    k = 8 * 5 + 3
    assert np.array_equal((by[:, 5] >> 3) & 1, (S[:, k] > 0).astype(np.uint8))
    # symmetric weights -> about half the bits set (5 sigma)
    ones = int((S > 0).sum())
    assert abs(ones - S.size / 2) < 5 * np.sqrt(S.size) / 2
    # mean / abs-mean against a plain python sum
    flat = [float(v) for v in c["W"].ravel()]
    assert abs(float(mu) - sum(flat) / len(flat)) < 1e-9
    assert abs(float(lam) - sum(abs(v) for v in flat) / len(flat)) < 1e-8


def test_sign_of_zero_and_constant_matrix():
    W = np.full((4, 32), -0.25, np.float32)
    mu, lam = O.weight_scales(W)
    assert mu == np.float32(-0.25) and lam == np.float32(0.25)
    assert np.all(O.binarize(W, mu) == 1)


# ---------------------------------------------------------------- I2: activations
def test_act_quant_range_and_error_bound():
    rng = np.random.default_rng(3)
    X = I.bf16_values((rng.standard_normal((64, 96)) * rng.lognormal(0, 2, (64, 1))).astype(np.float32))
    X[5] = 0.0
    q, gamma = O.act_quant(X)
    assert q.dtype == np.int8 and q.min() >= -128 and q.max() <= 127
    nz = np.abs(X).max(axis=1) > 0
    assert np.all(np.abs(q[nz].astype(int)).max(axis=1) >= 127)       # the amax element hits the top code
    assert np.all(q[5] == 0)
    err = np.abs(X.astype(np.float64) - q / gamma[:, None].astype(np.float64))
    bound = 0.5 / gamma.astype(np.float64) * (1 + 1e-5)   # slack: gamma itself is rounded to fp32
    clipped = (np.rint(X * gamma[:, None]) > 127)
    assert np.all(err[~clipped] <= np.broadcast_to(bound[:, None], err.shape)[~clipped])
    assert np.all(err[clipped] <= 2 * np.broadcast_to(bound[:, None], err.shape)[clipped])
    # gamma definition against python floats
    for t in (0, 7, 63):
        assert abs(float(gamma[t]) * float(np.abs(X[t]).max()) - 128.0) < 1e-4


# ---------------------------------------------------------------- I3, I4: 1-bit product
def test_onebit_gemm_bruteforce_and_parity():
    rng = np.random.default_rng(5)
    q = rng.integers(-128, 128, (5, 16)).astype(np.int8)
    S = rng.choice([-1, 1], (7, 16)).astype(np.int8)
    acc = O.onebit_gemm(q, S)
    for t, n in itertools.product(range(5), range(7)):
        assert acc[t, n] == sum(int(q[t, k]) * int(S[n, k]) for k in range(16))
    assert np.array_equal(acc % 2, (q.astype(int).sum(axis=1) % 2)[:, None] * np.ones((1, 7), int))
    assert np.all(np.abs(acc) <= np.abs(q.astype(int)).sum(axis=1)[:, None])
    # not transposed: a rectangular library product agrees
    assert np.array_equal(acc, q.astype(np.int64) @ S.astype(np.int64).T)


def test_onebit_layer_within_quantiser_error_of_exact_product():
    c = I.make_linear_case(32, 128, 48, 0, 0, seed=7, with_grad=False)
    f = O.linear_forward(c["X"], c["W"], beta=1.0)
    exact = float(f["lam"]) * (c["X"].astype(np.float64) @ f["S"].astype(np.float64).T)
    bound = float(f["lam"]) * (0.5 * 128 + 0.5) / f["gamma"].astype(np.float64)
    assert np.all(np.abs(f["y1"] - exact) <= bound[:, None] * (1 + 1e-9))
    # the bound is not vacuous: the product is far larger than the error
    assert np.abs(exact).mean() > 3 * np.abs(f["y1"] - exact).mean()


# ---------------------------------------------------------------- router + permutation
def test_router_fp32_order_close_to_fp64_and_softmax():
    c = I.make_linear_case(96, 512, 64, 16, 8, seed=9, with_grad=False)
    rt = O.router(c["X"], c["Wr"])
    assert np.allclose(rt["logits32"], rt["logits64"], rtol=0, atol=2e-5 * np.abs(rt["logits64"]).max())
    assert np.allclose(rt["probs"].sum(axis=1), 1.0)
    for t in (0, 50, 95):           # softmax against python floats
        l = [float(v) for v in rt["logits32"][t]]
        m = max(l)
        den = sum(np.exp(v - m) for v in l)
        assert abs(rt["gate"][t] - np.exp(l[rt["idx"][t]] - m) / den) < 1e-12
        assert rt["idx"][t] == l.index(m)
    # the planted Zipf assignment is what the router computes
    assert (rt["idx"] == c["planted"]).mean() > 0.98


def test_router_tie_goes_to_lowest_index():
    X = I.bf16_values(np.ones((3, 8), np.float32))
    Wr = I.bf16_values(np.array([[0.5] * 8, [1.0] * 8, [1.0] * 8, [0.25] * 8], np.float32))
    rt = O.router(X, Wr)
    assert np.all(rt["idx"] == 1)


def test_permutation_is_stable_sort():
    idx = np.array([2, 0, 1, 2, 0, 0, 3, 1], np.int32)
    perm, off = O.permutation(idx, 5)
    assert off.tolist() == [0, 3, 5, 7, 8, 8]
    assert perm.tolist() == [1, 4, 5, 2, 7, 0, 3, 6]


def test_zipf_quota_shares():
    ids = I.zipf_assignment(8192, 8, np.random.default_rng(0), True)
    share = np.bincount(ids, minlength=8) / 8192
    assert np.all(np.abs(share - I.zipf_shares(8)) < 5e-4)
    assert abs(I.zipf_shares(8)[0] - 0.398) < 2e-3


# ---------------------------------------------------------------- I5-I7: special cases of the layer
def _case(E, seed=21, T=40, K=64, N=48, r=16, **kw):
    return I.make_linear_case(T, K, N, r, E, seed=seed, **kw)


def test_hp_zeroed_gives_pure_onebit_layer():
    c = _case(1)
    pure = O.linear_forward(c["X"], c["W"], beta=c["beta"])
    for kw in (dict(A=np.zeros_like(c["A"]), B=c["B"]), dict(A=c["A"], B=np.zeros_like(c["B"])),
               dict(A=c["A"], B=c["B"], alpha=0.0)):
        kw.setdefault("alpha", c["alpha"])
        f = O.linear_forward(c["X"], c["W"], beta=c["beta"], **kw)
        assert np.array_equal(f["Y"], pure["Y"])
    # and the pure layer is beta * (lam/gamma) * S q written out by hand
    t, n = 3, 5
    s = sum(int(pure["q"][t, k]) * int(pure["S"][n, k]) for k in range(64))
    assert abs(pure["Y64"][t, n] - float(c["beta"][0]) * float(pure["lam"]) / float(pure["gamma"][t]) * s) < 1e-12


def test_all_experts_active_equals_dense_branch():
    c = _case(4, zipf=False)
    X, A, B = c["X"], c["A"], c["B"]
    E, r, K = A.shape
    N = B.shape[1]
    # unit gates: sum over experts == one dense branch of width E*r
    z_all = O.hp_branch_all_experts(X, A, B, np.ones((X.shape[0], E)))
    A_cat = A.reshape(E * r, K).astype(np.float64)
    B_cat = np.concatenate([B[e] for e in range(E)], axis=1).astype(np.float64)
    assert np.allclose(z_all, (X.astype(np.float64) @ A_cat.T) @ B_cat.T, rtol=1e-12, atol=1e-15)
    # softmax gates: dense branch with hidden block e scaled by p_e
    p = O.router(X, c["Wr"])["probs"]
    z_soft = O.hp_branch_all_experts(X, A, B, p)
    H = (X.astype(np.float64) @ A_cat.T) * np.repeat(p, r, axis=1)
    assert np.allclose(z_soft, H @ B_cat.T, rtol=1e-12, atol=1e-15)
    # routed top-1 picks exactly one of those terms
    rt = O.router(X, c["Wr"])
    _, z = O.hp_branch(X, A, B, rt["idx"])
    onehot = np.eye(E)[rt["idx"]]
    assert np.allclose(z, O.hp_branch_all_experts(X, A, B, onehot), rtol=1e-12, atol=1e-15)


def test_single_expert_has_unit_gate_and_dense_form():
    c = _case(1)
    f = O.linear_forward(c["X"], c["W"], c["A"], c["B"], None, c["alpha"], c["beta"])
    assert np.all(f["gate"] == 1.0) and np.all(f["idx"] == 0)
    dense = (c["X"].astype(np.float64) @ c["A"][0].astype(np.float64).T) @ c["B"][0].astype(np.float64).T
    assert np.allclose(f["Y64"], float(c["alpha"][0]) * dense + float(c["beta"][0]) * f["y1"], rtol=1e-12)
    g = O.linear_backward(c["dY"], c["X"], f, c["A"], c["B"], None, c["alpha"], c["beta"])
    assert "dWr" not in g


def test_routed_forward_sum_written_out_term_by_term():
    # Sec. 3.3 + Eq. 10-11 for a ROUTED layer, with python floats and plain loops only:
    #   Y[t,n] = alpha_n * p[t,e*] * (B_e* (A_e* x_t))[n] + beta_n * (lam / gamma_t) * sum_k S[n,k] q[t,k]
    # with e* the arg-max logit and p the softmax over all E logits.  Nothing of the oracle's forward is reused
    # except its quantised operands (q, gamma, S, lam), which have pins of their own above.
    T, K, N, r, E = 6, 32, 8, 4, 3
    c = I.make_linear_case(T, K, N, r, E, seed=61, zipf=False, scale_vector=True)
    c["Wr"] = I.bf16_values((c["Wr"] * 30).astype(np.float32))          # logits well apart: no near-tie, gates well below 1
    c["alpha"] = np.linspace(1.1, 1.9, N).astype(np.float32)
    c["beta"] = np.linspace(0.3, 0.7, N).astype(np.float32)
    f = O.linear_forward(c["X"], c["W"], c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    X, A, B, Wr = ([[float(v) for v in row] for row in m] if m.ndim == 2 else [[[float(v) for v in row] for row in e] for e in m]
                   for m in (c["X"], c["A"], c["B"], c["Wr"]))
    lam = float(f["lam"])

    def by_hand(use_gate=True, expert_shift=0, softmax_over_all=True):
        Y = [[0.0] * N for _ in range(T)]
        experts = []
        for t in range(T):
            logit = [sum(X[t][k] * Wr[e][k] for k in range(K)) for e in range(E)]
            best = max(range(E), key=lambda e: (logit[e], -e))
            m = max(logit)
            den = sum(np.exp(l - m) for l in logit) if softmax_over_all else np.exp(logit[best] - m)
            gate = np.exp(logit[best] - m) / den if use_gate else 1.0
            e = (best + expert_shift) % E
            experts.append(best)
            h = [sum(A[e][j][k] * X[t][k] for k in range(K)) for j in range(r)]
            for n in range(N):
                z = sum(B[e][n][j] * h[j] for j in range(r))
                acc = sum(int(f["S"][n, k]) * int(f["q"][t, k]) for k in range(K))
                Y[t][n] = float(c["alpha"][n]) * gate * z + float(c["beta"][n]) * (lam / float(f["gamma"][t])) * acc
        return np.array(Y), experts

    want, experts = by_hand()
    assert experts == f["idx"].tolist()
    assert len(set(experts)) > 1                                          # more than one expert is really in use
    assert 0.4 < float(f["gate"].min()) and float(f["gate"].max()) < 0.999   # the gate is not a disguised 1
    # the HP term is a visible share of the output, so an error in it cannot hide in the tolerance
    hp_share = np.abs(want - np.asarray(c["beta"], np.float64)[None, :] * f["y1"]).mean() / np.abs(want).mean()
    assert hp_share > 0.05
    tol = 1e-5 * np.abs(want).max()       # the oracle's gate comes from logits summed in fp32 order
    assert np.max(np.abs(f["Y64"] - want)) <= tol
    # planted mistakes: each one must break the same comparison
    for wrong in (by_hand(use_gate=False)[0], by_hand(expert_shift=1)[0], by_hand(softmax_over_all=False)[0]):
        assert np.max(np.abs(f["Y64"] - wrong)) > 100 * tol
    assert np.max(np.abs(f["Y64"] - (want - 2 * np.asarray(c["beta"], np.float64)[None, :] * f["y1"]))) > 100 * tol   # sign of the 1-bit term
    # and the stored output is that sum rounded once to bf16
    assert np.array_equal(f["Y"], O.round_to_bf16(f["Y64"]))


def test_bf16_rounding_helper():
    x = np.array([1.0, 1.00390625, 1.005859375, 1.01171875, -3.14159, 1e-3, 65504.0])
    r = O.round_to_bf16(x)
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == 1.0078125 and r[3] == 1.015625  # ties to even
    assert np.array_equal(r.astype(np.float32), I.bf16_values(x.astype(np.float32)))


# ---------------------------------------------------------------- I8: STE = exact gradient of the linear surrogate
def test_onebit_grads_are_gradients_of_linear_surrogate():
    c = _case(1, T=12, K=32, N=10, r=4, scale_vector=True)
    c["beta"] = np.linspace(0.2, 0.8, 10).astype(np.float32)
    f = O.linear_forward(c["X"], c["W"], beta=c["beta"])
    g = O.linear_backward(c["dY"], c["X"], f, beta=c["beta"])
    lam, S = float(f["lam"]), f["S"].astype(np.float64)
    xt = f["q"] / f["gamma"][:, None].astype(np.float64)
    dY = c["dY"].astype(np.float64)
    beta = c["beta"].astype(np.float64)

    def loss(xt_, Wq_):        # surrogate: beta * (xt @ Wq^T), Wq = lam*S treated as free
        return float((dY * (beta[None, :] * (xt_ @ Wq_.T))).sum())

    eps = 1e-3
    for (t, k) in [(0, 0), (5, 17), (11, 31)]:
        d = np.zeros_like(xt); d[t, k] = eps
        fd = (loss(xt + d, lam * S) - loss(xt - d, lam * S)) / (2 * eps)
        assert abs(fd - g["dX64"][t, k]) < 1e-9 * max(1, abs(fd))
    for (n, k) in [(0, 0), (4, 9), (9, 31)]:
        d = np.zeros_like(S); d[n, k] = eps
        fd = (loss(xt, lam * S + d) - loss(xt, lam * S - d)) / (2 * eps)
        assert abs(fd - g["dW"][n, k]) < 1e-9 * max(1, abs(fd))
    # dbeta: derivative w.r.t. each beta_n
    for n in (0, 7):
        d = np.zeros(10); d[n] = eps
        fd = (float((dY * ((beta + d)[None, :] * f["y1"])).sum()) - float((dY * ((beta - d)[None, :] * f["y1"])).sum())) / (2 * eps)
        assert abs(fd - g["dbeta"][n]) < 1e-9 * max(1, abs(fd))
    # inside the clip range the gradient w.r.t. X passes unchanged: dX == d(surrogate)/d(xt)
    assert np.allclose(g["dX64"], lam * (dY * beta[None, :]) @ S, rtol=1e-12)
    # shapes catch a transposed operand
    assert g["dW"].shape == c["W"].shape and g["dX64"].shape == c["X"].shape


# ---------------------------------------------------------------- I9: HP + router + alpha grads by finite differences
def test_hp_router_alpha_grads_finite_differences():
    c = _case(3, seed=33, T=10, K=32, N=12, r=4, zipf=False, scale_vector=True)
    c["Wr"] = I.bf16_values((c["Wr"] * 25).astype(np.float32))      # well separated logits
    c["alpha"] = np.linspace(1.2, 1.8, 12).astype(np.float32)
    X, W, A, B, Wr = c["X"], c["W"], c["A"], c["B"], c["Wr"]
    f = O.linear_forward(X, W, A, B, Wr, c["alpha"], c["beta"])
    g = O.linear_backward(c["dY"], X, f, A, B, Wr, c["alpha"], c["beta"])
    dY = c["dY"].astype(np.float64)
    idx = f["idx"]           # the top-1 choice is held fixed: it is piecewise constant

    def hp_loss(X_, A_, B_, Wr_, al_):
        # true forward of the HP branch with the 1-bit branch frozen; fp64 everywhere
        l = X_ @ Wr_.T
        p = np.exp(l - l.max(axis=1, keepdims=True)); p /= p.sum(axis=1, keepdims=True)
        gate = p[np.arange(len(idx)), idx]
        tot = 0.0
        for t in range(len(idx)):
            z = B_[idx[t]] @ (A_[idx[t]] @ X_[t])
            tot += float((dY[t] * al_ * gate[t] * z).sum())
        return tot

    X64, A64, B64, Wr64, al64 = (v.astype(np.float64) for v in (X, A, B, Wr, c["alpha"]))
    eps = 1e-5

    def fd(arr, pos, which):
        d = np.zeros_like(arr); d[pos] = eps
        args = dict(X_=X64, A_=A64, B_=B64, Wr_=Wr64, al_=al64)
        ap, am = dict(args), dict(args)
        ap[which] = arr + d; am[which] = arr - d
        return (hp_loss(**ap) - hp_loss(**am)) / (2 * eps)

    def close(a, b):
        return abs(a - b) <= 1e-4 * max(1e-3, abs(a))   # oracle gates come from the fp32-order logits

    for pos in [(0, 1, 5), (1, 3, 31), (2, 0, 0)]:
        assert close(fd(A64, pos, "A_"), g["dA"][pos])
    for pos in [(0, 11, 3), (1, 0, 0), (2, 5, 2)]:
        assert close(fd(B64, pos, "B_"), g["dB"][pos])
    for pos in [(0, 4), (1, 31), (2, 0)]:
        assert close(fd(Wr64, pos, "Wr_"), g["dWr"][pos])
    for pos in [(0,), (11,)]:
        assert close(fd(al64, pos, "al_"), g["dalpha"][pos[0]])
    # dX of the HP + router part = total dX minus the 1-bit part
    for pos in [(0, 0), (4, 13), (9, 31)]:
        assert close(fd(X64, pos, "X_"), g["dX64"][pos] - g["dX1"][pos])


# ---------------------------------------------------------------- I13: identities the fused kernels rely on
def test_reduction_identities():
    c = _case(3, seed=44, T=24, K=32, N=20, r=8, zipf=False)
    f = O.linear_forward(c["X"], c["W"], c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    g = O.linear_backward(c["dY"], c["X"], f, c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    dY = c["dY"].astype(np.float64)
    xt = f["q"] / f["gamma"][:, None].astype(np.float64)
    G = dY.T @ xt                                                   # un-scaled dW
    assert np.allclose(g["dbeta"], float(f["lam"]) * (f["S"] * G).sum(axis=1), rtol=1e-10)
    B64 = c["B"].astype(np.float64)
    dalpha = np.zeros(20)
    for e in range(3):
        sel = f["idx"] == e
        dB_raw = (dY[sel] * f["gate"][sel, None]).T @ f["h"][sel]
        dalpha += (B64[e] * dB_raw).sum(axis=1)
    assert np.allclose(g["dalpha"], dalpha, rtol=1e-10)
    al = float(c["alpha"][0])
    for t in (0, 13, 23):
        dH_raw = (al * dY[t]) @ B64[f["idx"][t]]
        assert abs(g["dg"][t] - float(f["h"][t] @ dH_raw)) < 1e-10 * max(1, abs(g["dg"][t]))


def test_decode_path_reads_packed_bits():
    c = _case(2, seed=55, T=4, K=64, N=32, r=8, with_grad=False)
    f = O.linear_forward(c["X"], c["W"], c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    d = O.decode_forward(c["X"], O.pack_bits(f["S"]), f["lam"], c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    assert np.array_equal(d["Y"], f["Y"]) and np.array_equal(d["acc"], f["acc"])


def test_library_matmul_special_case():
    torch = pytest.importorskip("torch")
    c = _case(1, T=16, K=64, N=24, r=8)
    f = O.linear_forward(c["X"], c["W"], c["A"], c["B"], None, c["alpha"], c["beta"])
    acc = torch.from_numpy(f["q"].astype(np.float64)) @ torch.from_numpy(f["S"].astype(np.float64)).T
    assert np.array_equal(acc.numpy().astype(np.int64), f["acc"])
    h = torch.from_numpy(c["X"].astype(np.float64)) @ torch.from_numpy(c["A"][0].astype(np.float64)).T
    assert np.allclose(h.numpy(), f["h"], rtol=1e-13)


def test_rmsnorm_closed_forms_and_library_routine():
    # App. A / Sec. 4.5: RMSNorm fused with the activation quantiser at inference.
    rng = np.random.default_rng(11)
    K = 384
    X = O.round_to_bf16(rng.standard_normal((5, K)) * 3.0)
    w = O.round_to_bf16(1.0 + 0.1 * rng.standard_normal(K))
    # constant rows: c / sqrt(c^2 + eps) * w
    for c in (0.5, -2.0, 8.0):
        y = O.rmsnorm(np.full((1, K), c), np.ones(K), 1e-6)
        assert np.allclose(y, c / np.sqrt(c * c + 1e-6), rtol=2.0 ** -8)
    # a power-of-two rescaling of the input changes nothing when eps = 0
    assert np.array_equal(O.rmsnorm(X, w, 0.0), O.rmsnorm(4.0 * X, w, 0.0))
    # unit mean square before the gain (within the bf16 rounding of the outputs)
    y1 = O.rmsnorm(X, np.ones(K), 0.0).astype(np.float64)
    assert np.allclose(np.mean(y1 * y1, axis=1), 1.0, rtol=2.0 ** -7)
    # the library routine in fp64, rounded to bf16, differs by at most one bf16 step
    import torch
    ref = torch.nn.functional.rms_norm(torch.from_numpy(np.asarray(X, np.float64)), (K,), torch.from_numpy(np.asarray(w, np.float64)), 1e-5).numpy()
    y = O.rmsnorm(X, w, 1e-5).astype(np.float64)
    assert np.all(np.abs(y - ref) <= 2.0 ** -7 * np.abs(ref) + 1e-30)
    # planted mistakes are caught by the same comparison: eps dropped into the wrong place, mean of |x| instead of x^2
    wrong1 = X / (np.sqrt(np.mean(X * X, axis=1, keepdims=True)) + 1e-1) * w
    wrong2 = X / np.mean(np.abs(X), axis=1, keepdims=True) * w
    for wrong in (wrong1, wrong2):
        assert not np.all(np.abs(wrong - ref) <= 2.0 ** -7 * np.abs(ref) + 1e-30)
    # every output is a bf16 value
    assert np.array_equal(O.round_to_bf16(y), y)


def test_decode_with_fused_norm_is_norm_then_decode():
    rng = np.random.default_rng(12)
    K, N = 128, 64
    X = O.round_to_bf16(rng.standard_normal((3, K)) * 2.0)
    w = O.round_to_bf16(1.0 + 0.2 * rng.standard_normal(K))
    W = rng.standard_normal((N, K)).astype(np.float32)
    mu, lam = O.weight_scales(W)
    bits = O.pack_bits(O.binarize(W, mu))
    a = O.decode_forward(X, bits, lam, norm_weight=w, norm_eps=1e-5)
    b = O.decode_forward(O.rmsnorm(X, w, 1e-5), bits, lam)
    assert np.array_equal(a["Y"], b["Y"]) and np.array_equal(a["q"], b["q"])
    c = O.decode_forward(X, bits, lam)
    assert not np.array_equal(a["q"], c["q"])


# ---------------------------------------------------------------- INT8 high-precision branch (Sec. 3.2)
@pytest.mark.parametrize("row", _golden("weight_quant"))
def test_weight_absmax_quant_worked(row):
    W = _mat(row[0])
    q, g = O.absmax_quant_matrix(W)
    assert g == np.float32(float(row[1].split()[1]))
    assert np.array_equal(q, _mat(row[2].split(None, 1)[1]).astype(np.int8))


@pytest.mark.parametrize("row", _golden("requant"))
def test_requant_hidden_worked(row):
    h = _mat(row[0]).astype(np.int64)
    qh, g = O.requant_hidden(h)
    assert g[0] == np.float32(float(row[1].split()[1]))       # 0.5, 1.5 -> 0, 2 (ties to even) in the second row: 3/8, 5/8 round to 0, 1
    assert np.array_equal(qh[0], np.array([int(v) for v in row[2].split()[1:]]))


def test_int8_expert_weights_range_and_error_bound():
    c = _case(3, zipf=False)
    A8, gA, B8, gB = O.quantize_experts(c["A"], c["B"])
    for W, W8, g in [(c["A"][e], A8[e], gA[e]) for e in range(3)] + [(c["B"][e], B8[e], gB[e]) for e in range(3)]:
        assert W8.dtype == np.int8 and W8.min() >= -128 and W8.max() <= 127
        assert np.abs(W8.astype(int)).max() >= 127                                  # the largest weight takes the top code
        assert abs(float(g) * float(np.abs(W).max()) - 128.0) < 1e-3
        err = np.abs(W.astype(np.float64) - W8 / np.float64(g))
        clipped = np.rint(W * g) > 127
        assert np.all(err[~clipped] <= 0.5 / g * (1 + 1e-5)) and np.all(err[clipped] <= 1.0 / g * (1 + 1e-5))


def test_int8_branch_bruteforce_and_scale():
    # every integer of the branch by python loops on a tiny routed case, and the real value it stands for
    T, K, N, r, E = 5, 16, 6, 4, 2
    c = I.make_linear_case(T, K, N, r, E, seed=71, zipf=False)
    c["Wr"] = I.bf16_values((c["Wr"] * 30).astype(np.float32))
    f = O.linear_forward(c["X"], c["W"], c["A"], c["B"], c["Wr"], c["alpha"], c["beta"], hp_int8=True)
    A8, gA, B8, gB = f["A8"], f["gA"], f["B8"], f["gB"]
    assert len(set(f["idx"].tolist())) == 2
    for t in range(T):
        e = int(f["idx"][t])
        h = [sum(int(A8[e, j, k]) * int(f["q"][t, k]) for k in range(K)) for j in range(r)]
        assert h == f["h_int"][t].tolist()
        amax = max(abs(v) for v in h)
        gh = np.float32(128.0) / np.float32(amax)
        assert gh == f["gamma_h"][t]
        qh = [int(np.clip(np.rint(np.float32(v) * gh), -128, 127)) for v in h]
        assert qh == f["qh"][t].tolist()
        for n in range(N):
            zi = sum(int(B8[e, n, j]) * qh[j] for j in range(r))
            assert zi == f["z_int"][t, n]
            real = zi / (float(gB[e]) * float(gh) * float(gA[e]) * float(f["gamma"][t]))
            assert abs(real - f["z"][t, n]) <= 1e-12 * max(1.0, abs(real))
            want = float(c["alpha"][0]) * f["gate"][t] * real + float(c["beta"][0]) * f["y1"][t, n]
            assert abs(want - f["Y64"][t, n]) <= 1e-12 * max(1.0, abs(want))


def test_int8_branch_within_quantiser_bound_of_the_fp_branch():
    # Sec. 4.6 (the FP16 ablation behaves like the INT8 branch): the INT8 result stays within the error bound the three
    # quantisers (activations, weights, hidden codes) allow around the un-quantised product B_e A_e x.
    c = _case(3, seed=23, T=48, K=128, N=40, r=16, zipf=False)
    f8 = O.linear_forward(c["X"], c["W"], c["A"], c["B"], c["Wr"], c["alpha"], c["beta"], hp_int8=True)
    ff = O.linear_forward(c["X"], c["W"], c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    assert np.array_equal(f8["idx"], ff["idx"])
    X = c["X"].astype(np.float64)
    idx = ff["idx"]
    gt = f8["gamma"].astype(np.float64)
    bound = np.zeros_like(ff["z"])
    for t in range(48):
        e = idx[t]
        A, B = c["A"][e].astype(np.float64), c["B"][e].astype(np.float64)
        dx, dA, dB = 1.0 / gt[t], 1.0 / float(f8["gA"][e]), 1.0 / float(f8["gB"][e])
        h_err = np.abs(A).sum(axis=1) * dx + dA * (np.abs(X[t]) + dx).sum() + 1.0 / (float(f8["gamma_h"][t]) * float(f8["gA"][e]) * gt[t])
        bound[t] = np.abs(B) @ h_err + dB * (np.abs(ff["h"][t]) + h_err).sum()
    err = np.abs(f8["z"] - ff["z"])
    assert np.all(err <= bound)
    assert np.sqrt(np.mean(err ** 2)) < 0.05 * np.sqrt(np.mean(ff["z"] ** 2))      # and in practice a few percent
    # planted mistakes break it: the hidden scale left out, the token's own scale left out
    wrong1 = f8["z_int"] / (f8["gB"].astype(np.float64)[idx] * f8["gA"].astype(np.float64)[idx] * gt)[:, None]
    wrong2 = f8["z_int"] / (f8["gB"].astype(np.float64)[idx] * f8["gA"].astype(np.float64)[idx] * f8["gamma_h"].astype(np.float64))[:, None]
    for wrong in (wrong1, wrong2):
        assert not np.all(np.abs(wrong - ff["z"]) <= bound)


def test_int8_branch_decode_uses_stored_codes():
    c = _case(2, seed=56, T=4, K=64, N=32, r=8, with_grad=False)
    f = O.linear_forward(c["X"], c["W"], c["A"], c["B"], c["Wr"], c["alpha"], c["beta"], hp_int8=True)
    stored = (f["A8"], f["gA"], f["B8"], f["gB"])
    d = O.decode_forward(c["X"], O.pack_bits(f["S"]), f["lam"], c["A"] * 0, c["B"] * 0, c["Wr"], c["alpha"], c["beta"], hp_int8=stored)
    assert np.array_equal(d["Y"], f["Y"]) and np.array_equal(d["z_int"], f["z_int"])


# ---------------------------------------------------------------- FFN-level decoupling (Eq. 11, Table 1)
def _ffn_case(T=12, Dm=32, F1=64, r=16, seed=81):
    rng = np.random.default_rng(seed)
    X = I.bf16_values(rng.standard_normal((T, Dm)).astype(np.float32))
    Wg, Wu = (rng.standard_normal((F1, Dm)) * 0.3).astype(np.float32), (rng.standard_normal((F1, Dm)) * 0.3).astype(np.float32)
    Wd = (rng.standard_normal((Dm, F1)) * 0.3).astype(np.float32)
    G = I.bf16_values((rng.standard_normal((r, Dm)) * 0.3).astype(np.float32))
    U = I.bf16_values((rng.standard_normal((r, Dm)) * 0.3).astype(np.float32))
    D = I.bf16_values((rng.standard_normal((Dm, r)) * 0.3).astype(np.float32))
    return X, Wg, Wu, Wd, G, U, D


def test_silu_reproducible_form_against_closed_values():
    x = np.array([0.0, 1.0, -1.0, 20.0, -20.0, 0.5], np.float32)
    want = [0.0, 1.0 / (1.0 + np.exp(-1.0)), -1.0 / (1.0 + np.exp(1.0)), 20.0, -20.0 * np.exp(-20.0) / (1 + np.exp(-20.0)), 0.5 / (1.0 + np.exp(-0.5))]
    got = O.silu_fp32(x)
    assert got.dtype == np.float32
    assert np.allclose(got, want, rtol=2e-7, atol=1e-12)
    assert got[1] + (-got[2]) == np.float32(1.0) or abs(float(got[1]) - float(got[2]) - 1.0) < 1e-6     # silu(x) - silu(-x) = x


def test_ffn_decoupled_term_by_term():
    # Eq. 11 on a tiny case with python floats: the 1-bit FFN as three hand-evaluated 1-bit linears, the INT8 FFN from
    # its integers; planted mistakes (branch scales swapped, activation on the wrong operand, un-gated form) are caught
    X, Wg, Wu, Wd, G, U, D = _ffn_case()
    f = O.ffn_decoupled_forward(X, Wg, Wu, Wd, G, U, D, alpha=2.0, beta=0.2)
    T, Dm = X.shape
    F1, r = Wg.shape[0], G.shape[0]

    def onebit(Xin, W):          # Eq. 3-10 by hand: fp32 scale decisions come from the pinned helpers, sums are python ints
        mu, lam = O.weight_scales(W)
        S = O.binarize(W, mu)
        q, gam = O.act_quant(Xin)
        out = [[float(lam) / float(gam[t]) * sum(int(S[n, k]) * int(q[t, k]) for k in range(Xin.shape[1])) for n in range(W.shape[0])]
               for t in range(Xin.shape[0])]
        return np.array(out), q, gam

    g1, q, gam = onebit(X, Wg)
    u1, _, _ = onebit(X, Wu)
    g1b, u1b = O.round_to_bf16(g1), O.round_to_bf16(u1)
    assert np.array_equal(g1b, f["gate"]["Y"]) and np.array_equal(u1b, f["up"]["Y"])
    m1 = O.round_to_bf16(np.array([[g1b[t, j] / (1.0 + np.exp(-g1b[t, j])) * u1b[t, j] for j in range(F1)] for t in range(T)]))
    y1, _, _ = onebit(m1.astype(np.float32), Wd)
    G8, gG = O.absmax_quant_matrix(G); U8, gU = O.absmax_quant_matrix(U); D8, gD = O.absmax_quant_matrix(D)

    def int8_ffn(act_on="gate", gated=True):
        z = np.zeros((T, Dm))
        for t in range(T):
            gi = [sum(int(G8[j, k]) * int(q[t, k]) for k in range(Dm)) for j in range(r)]
            ui = [sum(int(U8[j, k]) * int(q[t, k]) for k in range(Dm)) for j in range(r)]
            assert gi == f["hp"]["g_int"][t].tolist() and ui == f["hp"]["u_int"][t].tolist()
            g = [v / (float(gG) * float(gam[t])) for v in gi]
            u = [v / (float(gU) * float(gam[t])) for v in ui]
            a, b = (g, u) if act_on == "gate" else (u, g)
            m = [a[j] / (1.0 + np.exp(-a[j])) * (b[j] if gated else 1.0) for j in range(r)]
            amax = max(abs(v) for v in m)
            codes = [int(np.clip(np.rint(v * 128.0 / amax), -128, 127)) for v in m]
            for n in range(Dm):
                z[t, n] = sum(int(D8[n, j]) * codes[j] for j in range(r)) / (float(gD) * 128.0 / amax)
        return z

    z = int8_ffn()
    # codes decided in fp32 by the oracle may differ by one from the python-float decision at a rounding boundary: the
    # real-valued z is compared within one code's worth
    tol = np.abs(D8.astype(np.float64)).sum(axis=1)[None, :] * 1.01 / (float(gD) * f["hp"]["gamma_m"].astype(np.float64))[:, None]
    assert np.all(np.abs(z - f["hp"]["z"]) <= tol)
    want = 2.0 * z + 0.2 * y1
    err = np.abs(f["Y64"] - want)
    assert np.all(err <= 2.0 * tol + 1e-9)
    scale = np.abs(want).mean()
    assert err.mean() < 0.02 * scale
    for wrong in (0.2 * z + 2.0 * y1, 2.0 * int8_ffn(act_on="up") + 0.2 * y1, 2.0 * int8_ffn(gated=False) + 0.2 * y1, 2.0 * z - 0.2 * y1):
        assert np.abs(f["Y64"] - wrong).mean() > 0.1 * scale
    assert np.array_equal(f["Y"], O.round_to_bf16(f["Y64"]))


def test_ffn_decoupled_special_cases():
    X, Wg, Wu, Wd, G, U, D = _ffn_case(seed=82)
    f = O.ffn_decoupled_forward(X, Wg, Wu, Wd, G, U, D, alpha=0.0, beta=1.0)
    # alpha = 0: the plain 1-bit FFN, i.e. three pure 1-bit linears around the gate
    assert np.array_equal(f["Y"], O.round_to_bf16(f["down"]["y1"]))
    # beta = 0: the INT8 FFN alone, within the quantisers' reach of the un-quantised gated FFN of width r
    f8 = O.ffn_decoupled_forward(X, Wg, Wu, Wd, G, U, D, alpha=1.0, beta=0.0)
    X64 = X.astype(np.float64)
    g, u = X64 @ G.astype(np.float64).T, X64 @ U.astype(np.float64).T
    ref = (g / (1.0 + np.exp(-g)) * u) @ D.astype(np.float64).T
    rel = np.sqrt(np.mean((f8["Y64"] - ref) ** 2)) / np.sqrt(np.mean(ref ** 2))
    assert rel < 0.05
    # the codes of the hidden activation use the full range and the same quantiser as activations
    assert np.all(np.abs(f8["hp"]["qm"].astype(int)).max(axis=1) >= 127)
