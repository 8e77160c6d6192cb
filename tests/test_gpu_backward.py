"""GPU parity tests (backward side): straight-through gradients of the layer
through the C ABI against the CPU oracle (App. B.1)."""
import numpy as np
import pytest
import torch

from oracle import pquant_oracle as O
from paper_2602_22592_b200 import binding as pqb
from paper_2602_22592_b200 import inputs as I
from paper_2602_22592_b200.layer import PQLinear
from test_gpu_forward import CASES, STRICT, TOL_BF16, TOL_RMS, check_status, f32, rel_err, rms_err

pytestmark = pytest.mark.gpu


def run_fwd_bwd(c, scale_vector):
    L = PQLinear(c["T"], c["K"], c["N"], c["r"], c["E"], scale_vector=scale_vector).load_case(c)
    L.pack()
    L.forward()
    L.backward()
    torch.cuda.synchronize()
    check_status()
    return L


TOL_DL = 3e-2   # router-logit gradient (an intermediate, not an output): dg is a near-cancelling sum over the hidden width


def check_backward(c, L, f, g, scale_vector):
    """Every gradient three ways: element-wise with the rms floor (<= 2e-2), as a whole tensor (<= 5e-3 of its
    norm, which a dropped contribution cannot pass), and -- where no bf16 intermediate is involved -- element-wise
    with the strict floor of 1e-2 rms."""
    red = (lambda v: v) if scale_vector else (lambda v: np.array([v.sum()]))
    pairs = {"dX": (f32(L.dX), g["dX"]), "dW": (f32(L.dW), g["dW"]), "dbeta": (f32(L.dbeta), red(g["dbeta"]))}
    strict = []
    routed = c["r"] > 0 and c["E"] > 1
    if not routed and not scale_vector:
        # with routing dX carries the bf16-rounded logit gradient and dH / c; with per-feature scales the sign
        # matrix enters the dX product as bf16(beta_n) S
        strict.append("dX")
    if c["r"] > 0:
        pairs["dA"] = (f32(L.dA), g["dA"])
        pairs["dB"] = (f32(L.dB), g["dB"])
        pairs["dalpha"] = (f32(L.dalpha), red(g["dalpha"]))
        strict += ["dB", "dalpha"]
        if routed:
            pairs["dWr"] = (f32(L.dWr), g["dWr"])
    errs = {k: rel_err(a, b) for k, (a, b) in pairs.items()}
    bad = {k: v for k, v in errs.items() if not v <= TOL_BF16}
    assert not bad, f"gradients outside tolerance: {bad} (all: {errs})"
    # (a scalar feature scale's gradient is one near-cancelling sum over all tokens and features: for it the two
    # measures coincide and the element-wise tolerance is the one that applies)
    whole = {k: rms_err(a, b) for k, (a, b) in pairs.items() if np.size(b) > 1}
    bad = {k: v for k, v in whole.items() if not v <= TOL_RMS}
    assert not bad, f"whole-tensor error too large: {bad} (all: {whole})"
    tight = {k: rel_err(*pairs[k], STRICT) for k in strict}
    bad = {k: v for k, v in tight.items() if not v <= TOL_BF16}
    assert not bad, f"outside tolerance at the strict floor: {bad}"
    if routed:
        # the logit gradient the kernels leave in the workspace, in sorted token order
        perm = L.saved_view()["perm"].cpu().numpy()
        dl = f32(L.bwd_view()["dl"])
        assert rel_err(dl, g["dl"][perm]) <= TOL_DL and rms_err(dl, g["dl"][perm]) <= TOL_RMS
    return errs


BWD_CASES = dict(CASES)
BWD_CASES["routed8_vec"] = dict(T=700, K=512, N=512, r=64, E=8, scale_vector=True, alpha=1.3, beta=0.6)


@pytest.mark.parametrize("name", list(BWD_CASES))
def test_backward_matches_oracle(name):
    kw = dict(BWD_CASES[name])
    sv = kw.pop("scale_vector", False)
    c = I.make_linear_case(kw.pop("T"), kw.pop("K"), kw.pop("N"), kw.pop("r"), kw.pop("E"), seed=11, scale_vector=sv, **kw)
    if sv:   # distinct per-feature scales so that a misplaced index shows
        c["alpha"] = (c["alpha"] * np.linspace(0.8, 1.2, c["N"])).astype(np.float32)
        c["beta"] = (c["beta"] * np.linspace(1.2, 0.8, c["N"])).astype(np.float32)
    f = O.linear_forward(c["X"], c["W"], c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    g = O.linear_backward(c["dY"], c["X"], f, c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    L = run_fwd_bwd(c, sv)
    check_backward(c, L, f, g, sv)


def test_backward_empty_experts_and_zero_beta():
    # experts 1 and 3 receive no token: their gradients must be exactly zero;
    # beta = 0 switches the 1-bit input gradient off without dividing by zero
    c = I.make_linear_case(300, 256, 256, 32, 4, seed=9, zipf=False, beta=0.0)
    c["X"][7] = 0.0
    c["Wr"][:] = 0.0
    c["Wr"][2] = I.bf16_values(np.full(256, 0.5, np.float32))
    c["X"] = I.bf16_values(np.abs(c["X"]))
    f = O.linear_forward(c["X"], c["W"], c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    g = O.linear_backward(c["dY"], c["X"], f, c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    L = run_fwd_bwd(c, False)
    assert torch.all(L.dA[1] == 0) and torch.all(L.dA[3] == 0) and torch.all(L.dB[1] == 0) and torch.all(L.dB[3] == 0)
    assert torch.all(L.dW == 0)
    errs = {k: rel_err(f32(getattr(L, k)), g[k]) for k in ("dX", "dA", "dB", "dWr")}
    assert all(v <= TOL_BF16 for v in errs.values()), errs


def _dx_terms(c, g):
    """The three contributions to dX from the oracle's pieces: 1-bit, HP, router (App. B.1, Sec. 3.3)."""
    dX3 = g["dl"] @ c["Wr"].astype(np.float64) if "dl" in g else np.zeros_like(g["dX64"])
    return g["dX1"], g["dX64"] - g["dX1"] - dX3, dX3


def test_backward_hp_term_of_dx_alone():
    # beta = 0 removes the 1-bit term, a zero router matrix removes the router term (uniform gates, expert 0 for
    # every token): dX is the HP term A_e^T dH alone, and is checked as a whole tensor
    c = I.make_linear_case(520, 512, 384, 64, 4, seed=61, zipf=False, beta=0.0)
    c["Wr"][:] = 0.0
    f = O.linear_forward(c["X"], c["W"], c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    g = O.linear_backward(c["dY"], c["X"], f, c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    d1, d2, d3 = _dx_terms(c, g)
    assert not np.any(d1) and not np.any(d3) and np.any(d2)
    assert np.allclose(f["gate"], 0.25) and not np.any(f["idx"])
    L = run_fwd_bwd(c, False)
    assert rel_err(f32(L.dX), g["dX"]) <= TOL_BF16 and rms_err(f32(L.dX), g["dX"]) <= TOL_RMS
    assert np.any(g["dl"]) and rms_err(f32(L.dWr), g["dWr"]) <= TOL_RMS      # the router still gets its gradient


def test_backward_router_term_of_dx_isolated():
    # beta = 0 and a natural (unplanted) router: gates far from 1, so the router term dl . Wr is a large share of
    # dX.  What the GPU adds on top of the oracle's HP term must be the oracle's router term.
    c = I.make_linear_case(640, 512, 384, 32, 8, seed=62, zipf=False, beta=0.0)
    c["Wr"] = I.bf16_values((c["Wr"] * 4).astype(np.float32))
    f = O.linear_forward(c["X"], c["W"], c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    g = O.linear_backward(c["dY"], c["X"], f, c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    d1, d2, d3 = _dx_terms(c, g)
    share = np.sqrt(np.mean(d3 ** 2)) / np.sqrt(np.mean(g["dX64"] ** 2))
    assert not np.any(d1) and share > 0.25
    L = run_fwd_bwd(c, False)
    check_backward(c, L, f, g, False)
    assert rms_err(f32(L.dX).astype(np.float64) - d2, d3) <= 4 * TOL_RMS / share


def test_backward_is_deterministic():
    c = I.make_linear_case(512, 512, 512, 64, 4, seed=3)
    L = run_fwd_bwd(c, False)
    keep = [t.clone() for t in (L.dX, L.dW, L.dA, L.dB, L.dWr, L.dalpha, L.dbeta)]
    L.backward()
    torch.cuda.synchronize()
    for a, b in zip(keep, (L.dX, L.dW, L.dA, L.dB, L.dWr, L.dalpha, L.dbeta)):
        assert torch.equal(a, b)


def _all_outputs(L):
    names = ("Y", "dX", "dW", "dA", "dB", "dWr", "dalpha", "dbeta")
    return [getattr(L, n).clone() for n in names if getattr(L, n, None) is not None]


@pytest.mark.parametrize("E", [1, 4])
def test_helper_stream_changes_no_bit(E):
    # the helper stream only reorders independent kernels: results are bit-identical with it on or off
    c = I.make_linear_case(777, 512, 640, 64, E, seed=21)
    L = run_fwd_bwd(c, False)
    on = _all_outputs(L)
    pqb.pq_set_option(pqb.PQ_OPT_SIDE_STREAM, 0)
    try:
        L.forward()
        L.backward()
        torch.cuda.synchronize()
        off = _all_outputs(L)
    finally:
        pqb.pq_set_option(pqb.PQ_OPT_SIDE_STREAM, 1)
    check_status()
    for a, b in zip(on, off):
        assert torch.equal(a, b)


def test_helper_stream_under_graph_capture():
    # a captured forward + backward holds the fork to the helper stream and the join as graph edges;
    # replays match the eager call bit for bit
    c = I.make_linear_case(640, 512, 512, 32, 1, seed=22)
    L = run_fwd_bwd(c, False)      # eager run: creates the helper stream outside the capture
    want = _all_outputs(L)
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        L.forward()
        L.backward()
        torch.cuda.synchronize()
        with torch.cuda.graph(g, stream=s):
            L.forward()
            L.backward()
    for t in (L.Y, L.dX, L.dW, L.dA, L.dB, L.dalpha, L.dbeta):
        t.zero_()
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    check_status()
    for a, b in zip(want, _all_outputs(L)):
        assert torch.equal(a, b)


@pytest.mark.parametrize("K,N,E,r", [(2048, 5632, 1, 128), (2048, 5632, 8, 128), (5632, 2048, 8, 128), (2048, 2048, 8, 128),
                                     (2048, 2048, 0, 0)])
def test_full_size_projection_on_sampled_tokens(K, N, E, r):
    # The 1.3B projections in the launch configuration the benchmark times (8192 tokens): up / gate, down, the
    # attention-shaped 2048 -> 2048 linear with 8 experts, and the same as a pure 1-bit linear (the paper's attention
    # form) -- too large for the oracle as a whole.  Every per-token quantity depends on its own row of X only and every
    # weight gradient is a sum over tokens, so with dY zero outside a sample of rows the oracle on the sampled rows alone
    # gives Y and dX of those rows and ALL of dW, dA, dB, dWr, dalpha, dbeta; dX of the other rows must be zero.
    T = 8192
    c = I.make_linear_case(T, K, N, r, E, seed=31)
    rows = np.sort(np.random.default_rng(5).choice(T, 96, replace=False))
    dY = np.zeros_like(c["dY"])
    dY[rows] = c["dY"][rows]
    c["dY"] = dY
    L = run_fwd_bwd(c, False)
    f = O.linear_forward(c["X"][rows], c["W"], c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    g = O.linear_backward(dY[rows], c["X"][rows], f, c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    # integers of the sampled rows: codes, gamma, expert choice
    sv = L.saved_view()
    pos = sv["pos"].cpu().numpy()[rows]
    assert np.array_equal(sv["q"].cpu().numpy()[pos], f["q"])
    assert np.array_equal(f32(sv["gamma"])[pos], f["gamma"])
    if E > 1:
        assert np.array_equal(sv["expert"].cpu().numpy()[rows], f["idx"])
    pairs = {"Y": (f32(L.Y)[rows], f["Y"]), "dX": (f32(L.dX)[rows], g["dX"]), "dW": (f32(L.dW), g["dW"]),
             "dbeta": (f32(L.dbeta), np.array([g["dbeta"].sum()]))}
    others = np.ones(T, bool)
    others[rows] = False
    assert not np.any(f32(L.dX)[others])
    if r > 0:
        pairs["dA"] = (f32(L.dA), g["dA"])
        pairs["dB"] = (f32(L.dB), g["dB"])
        pairs["dalpha"] = (f32(L.dalpha), np.array([g["dalpha"].sum()]))
    if E > 1:
        pairs["dWr"] = (f32(L.dWr), g["dWr"])
    errs = {k: rel_err(a, b) for k, (a, b) in pairs.items()}
    bad = {k: v for k, v in errs.items() if not v <= TOL_BF16}
    assert not bad, f"outside tolerance: {bad} (all: {errs})"
    whole = {k: rms_err(a, b) for k, (a, b) in pairs.items() if np.size(b) > 1}
    bad = {k: v for k, v in whole.items() if not v <= TOL_RMS}
    assert not bad, f"whole-tensor error too large: {bad} (all: {whole})"


def test_first_use_inside_a_capture_keeps_plain_stream_order():
    # a stream whose first call is made while it is being captured gets no helper stream (nothing is created
    # during a capture): the graph holds the kernels in plain order and replays to the same bits
    c = I.make_linear_case(384, 256, 320, 32, 1, seed=23)
    L = run_fwd_bwd(c, False)
    want = _all_outputs(L)
    s = torch.cuda.Stream()            # never used with the library before
    s.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        with torch.cuda.graph(g, stream=s):
            L.forward()
            L.backward()
    for t in (L.Y, L.dX, L.dW, L.dA, L.dB, L.dalpha, L.dbeta):
        t.zero_()
    g.replay()
    torch.cuda.synchronize()
    check_status()
    for a, b in zip(want, _all_outputs(L)):
        assert torch.equal(a, b)
    with torch.cuda.stream(s):         # after the capture the stream gets its helper as usual
        L.forward()
        L.backward()
    torch.cuda.synchronize()
    for a, b in zip(want, _all_outputs(L)):
        assert torch.equal(a, b)


@pytest.mark.parametrize("T", [1, 3, 33, 130])
def test_few_tokens_routed(T):
    # fewer tokens than a router warp group, a block or a tile holds; most experts stay empty
    c = I.make_linear_case(T, 256, 256, 32, 8, seed=40 + T, zipf=False)
    f = O.linear_forward(c["X"], c["W"], c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    g = O.linear_backward(c["dY"], c["X"], f, c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    L = run_fwd_bwd(c, False)
    sv = L.saved_view()
    assert np.array_equal(sv["expert"].cpu().numpy(), f["idx"])
    assert np.array_equal(sv["perm"].cpu().numpy(), f["perm"])
    assert rel_err(f32(L.Y), f["Y"]) <= TOL_BF16
    check_backward(c, L, f, g, False)


@pytest.mark.parametrize("shape", [dict(T=333, K=384, N=544, r=64, E=1), dict(T=1000, K=512, N=768, r=128, E=8),
                                   dict(T=200, K=256, N=320, r=0, E=0), dict(T=200, K=4096, N=64, r=16, E=4),
                                   dict(T=70, K=8704, N=64, r=0, E=0)])
def test_training_path_with_fused_rmsnorm(shape):
    # App. A: RMSNorm fused in front of the quantiser, training-size path.  X is un-normalised (rows stretched by very
    # different factors); codes, scales and routing must equal the oracle's norm-then-layer exactly, the gradients are
    # those with respect to the normalised activation.
    c = I.make_linear_case(shape["T"], shape["K"], shape["N"], shape["r"], shape["E"], seed=27)
    rng = np.random.default_rng(6)
    c["X"] = I.bf16_values(c["X"] * rng.uniform(0.25, 6.0, size=(c["T"], 1)).astype(np.float32))
    w = I.bf16_values(1.0 + 0.1 * rng.standard_normal(c["K"]).astype(np.float32))
    eps = 1e-5
    Xn = O.rmsnorm(c["X"], w, eps)
    f = O.linear_forward(Xn, c["W"], c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    g = O.linear_backward(c["dY"], Xn, f, c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    L = PQLinear(c["T"], c["K"], c["N"], c["r"], c["E"], fused_rmsnorm=True, guard=True).load_case(c)
    L.norm_weight = torch.from_numpy(w).to(L.X.device).to(torch.bfloat16)
    L.norm_eps = eps
    L.pack()
    L.forward()
    L.backward()
    torch.cuda.synchronize()
    check_status()
    assert L.check_guards() == 0
    sv = L.saved_view()
    perm = sv["perm"].cpu().numpy()
    assert np.array_equal(sv["q"].cpu().numpy(), f["q"][perm])
    assert np.array_equal(f32(sv["gamma"]), f["gamma"][perm])
    assert np.array_equal(f32(sv["xs"]), Xn[perm])                      # the normalised activation, bit for bit
    if c["E"] > 1:
        assert np.array_equal(sv["expert"].cpu().numpy(), f["idx"])
    assert rel_err(f32(L.Y), f["Y"]) <= TOL_BF16 and rms_err(f32(L.Y), f["Y"]) <= TOL_RMS
    check_backward(c, L, f, g, False)
    # and it is not the layer applied to the un-normalised input
    f_raw = O.linear_forward(c["X"], c["W"], c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    assert not np.array_equal(f_raw["q"], f["q"])


def test_fused_rmsnorm_flag_and_arguments_must_agree():
    c = I.make_linear_case(128, 64, 64, 32, 1, seed=1)
    L = PQLinear(128, 64, 64, 32, 1).load_case(c)           # desc without the flag
    L.pack()
    w = torch.ones(64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(pqb.PqError) as ei:
        pqb.pq_linear_forward_rms(L.desc, L.X, w, 1e-5, L.w_s8, L.w_scales, L.A, L.B, None, L.alpha, L.beta, L.Y, L.saved, L.ws_fwd)
    assert ei.value.status == pqb.PQ_ERR_NULL
