"""GPU parity tests of the decode path (App. A): a few tokens against the packed sign bits,
through the C ABI, against the CPU oracle reading the same bits back."""
import numpy as np
import pytest
import torch

from oracle import pquant_oracle as O
from paper_2602_22592_b200 import binding as pqb
from paper_2602_22592_b200 import inputs as I
from paper_2602_22592_b200.layer import PQLinear
from test_gpu_forward import TOL_BF16, check_status, f32, rel_err

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True, params=["stream", "stream_dp4a", "stream_mma", "pair"])
def decode_kernels(request):
    """Every test runs on the streaming kernel (weights in its own layout; bit product as the library picks it, on dp4a
    only, on the tensor cores only) and on the two-kernel path."""
    stream = request.param != "pair"
    PQLinear.stream_decode = stream
    pqb.pq_set_option(pqb.PQ_OPT_DECODE_STREAM, 2 if stream else 0)   # 2: also for one small linear
    pqb.pq_set_option(pqb.PQ_OPT_DECODE_MMA_FROM, {"stream_dp4a": 17, "stream_mma": 1}.get(request.param, 5))
    # the forced variants also walk the two work lists side by side (two halves of a CTA), the plain one in turn
    pqb.pq_set_option(pqb.PQ_OPT_DECODE_INTERLEAVE, 2 if request.param in ("stream_dp4a", "stream_mma") else 0)
    yield request.param
    pqb.pq_set_option(pqb.PQ_OPT_DECODE_INTERLEAVE, 1)
    PQLinear.stream_decode = True
    pqb.pq_set_option(pqb.PQ_OPT_DECODE_STREAM, 1)
    pqb.pq_set_option(pqb.PQ_OPT_DECODE_MMA_FROM, 5)


def run_decode(c, scale_vector=False):
    L = PQLinear(c["T"], c["K"], c["N"], c["r"], c["E"], scale_vector=scale_vector, training=False, dump_acc=True).load_case(c)
    L.pack(bits_only=True)
    L.decode()
    torch.cuda.synchronize()
    check_status()
    return L


def check_decode(c, L):
    mu, lam = O.weight_scales(c["W"])
    bits = O.pack_bits(O.binarize(c["W"], mu))
    assert np.array_equal(L.w_bits.cpu().numpy().view(np.uint32), bits)
    f = O.decode_forward(c["X"], bits, lam, c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    v = L.decode_view()
    # integers: router index, int8 codes (through their sum), the 1-bit product itself
    assert np.array_equal(v["expert"].cpu().numpy(), f["idx"])
    assert np.array_equal(f32(v["gamma"]), f["gamma"])
    assert np.array_equal(v["code_sum"].cpu().numpy(), f["q"].astype(np.int64).sum(axis=1))
    assert np.array_equal(v["acc"].cpu().numpy().astype(np.int64), f["acc"])
    assert rel_err(f32(v["gate"]), f["gate"]) <= 1e-5
    assert rel_err(f32(L.Y), f["Y"]) <= TOL_BF16
    return f


DECODE_CASES = {
    "m1_small": dict(T=1, K=256, N=96, r=32, E=4),
    "m5_odd_words": dict(T=5, K=2080, N=992, r=40, E=3),          # 65 weight words per row, r not a multiple of 32
    "m16_two_groups": dict(T=16, K=512, N=2048, r=64, E=8),
    "m9_dense_hp": dict(T=9, K=384, N=320, r=160, E=1),
    "m3_pure_1bit": dict(T=3, K=1024, N=64, r=0, E=0),
    "m12_vector_scales": dict(T=12, K=320, N=4736, r=16, E=2, scale_vector=True, alpha=1.5, beta=0.4),
    "m2_widest_hp": dict(T=2, K=512, N=288, r=256, E=2),           # the widest branch the decode path takes
}


@pytest.mark.parametrize("name", list(DECODE_CASES))
def test_decode_matches_oracle(name):
    kw = dict(DECODE_CASES[name])
    sv = kw.pop("scale_vector", False)
    c = I.make_linear_case(kw.pop("T"), kw.pop("K"), kw.pop("N"), kw.pop("r"), kw.pop("E"), seed=21, scale_vector=sv,
                           exact_quota=False, with_grad=False, **kw)
    if sv:
        c["alpha"] = (c["alpha"] * np.linspace(0.8, 1.2, c["N"])).astype(np.float32)
        c["beta"] = (c["beta"] * np.linspace(1.2, 0.8, c["N"])).astype(np.float32)
    check_decode(c, run_decode(c, sv))


@pytest.mark.parametrize("M", [1, 4, 16])
@pytest.mark.parametrize("proj", [0, 2])
def test_decode_3b_shapes(M, proj):
    # the 3B-shaped layers the decode benchmark streams: 3200 -> 8640 (gate) and 8640 -> 3200 (down)
    c = I.config_decode(M, seed=4)[proj]
    check_decode(c, run_decode(c))


@pytest.mark.parametrize("name", ["m1_small", "m5_odd_words", "m16_two_groups", "m12_vector_scales", "m3_pure_1bit"])
def test_decode_with_fused_rmsnorm(name):
    # App. A: RMSNorm fused in front of the activation quantiser.  X is the un-normalised activation (here the case's
    # tokens stretched row by row); codes, routing and the 1-bit sums must still agree exactly with the oracle.
    kw = dict(DECODE_CASES[name])
    scale_vector = kw.pop("scale_vector", False)
    c = I.make_linear_case(kw.pop("T"), kw.pop("K"), kw.pop("N"), kw.pop("r"), kw.pop("E"), seed=31, exact_quota=False, with_grad=False,
                           scale_vector=scale_vector, **kw)
    rng = np.random.default_rng(5)
    c["X"] = I.bf16_values(c["X"] * rng.uniform(0.25, 6.0, size=(c["T"], 1)).astype(np.float32))
    w = I.bf16_values(1.0 + 0.1 * rng.standard_normal(c["K"]).astype(np.float32))
    eps = 1e-5
    L = PQLinear(c["T"], c["K"], c["N"], c["r"], c["E"], scale_vector=scale_vector, training=False, dump_acc=True).load_case(c)
    L.norm_weight = torch.from_numpy(w).to(L.X.device).to(torch.bfloat16)
    L.norm_eps = eps
    L.pack(bits_only=True)
    L.decode()
    torch.cuda.synchronize()
    check_status()
    mu, lam = O.weight_scales(c["W"])
    bits = O.pack_bits(O.binarize(c["W"], mu))
    f = O.decode_forward(c["X"], bits, lam, c["A"], c["B"], c["Wr"], c["alpha"], c["beta"], norm_weight=w, norm_eps=eps)
    v = L.decode_view()
    assert np.array_equal(v["expert"].cpu().numpy(), f["idx"])
    assert np.array_equal(f32(v["gamma"]), f["gamma"])
    assert np.array_equal(v["code_sum"].cpu().numpy(), f["q"].astype(np.int64).sum(axis=1))
    assert np.array_equal(v["acc"].cpu().numpy().astype(np.int64), f["acc"])
    assert rel_err(f32(L.Y), f["Y"]) <= TOL_BF16
    # and it is not the un-normalised result
    g = O.decode_forward(c["X"], bits, lam, c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    assert not np.array_equal(g["q"], f["q"])


def test_fused_rmsnorm_zero_token_and_bad_epsilon():
    c = I.make_linear_case(3, 256, 96, 32, 4, seed=33, exact_quota=False, with_grad=False)
    c["X"][1, :] = 0.0                                  # an all-zero token: normalised to zeros, codes all zero
    w = I.bf16_values(np.linspace(0.5, 1.5, c["K"]).astype(np.float32))
    L = PQLinear(c["T"], c["K"], c["N"], c["r"], c["E"], training=False, dump_acc=True).load_case(c)
    L.norm_weight = torch.from_numpy(w).to(L.X.device).to(torch.bfloat16)
    L.norm_eps = 1e-6
    L.pack(bits_only=True)
    L.decode()
    torch.cuda.synchronize()
    check_status()
    mu, lam = O.weight_scales(c["W"])
    bits = O.pack_bits(O.binarize(c["W"], mu))
    f = O.decode_forward(c["X"], bits, lam, c["A"], c["B"], c["Wr"], c["alpha"], c["beta"], norm_weight=w, norm_eps=1e-6)
    v = L.decode_view()
    assert np.array_equal(v["acc"].cpu().numpy().astype(np.int64), f["acc"])
    assert int(v["code_sum"][1]) == 0 and np.array_equal(f32(v["gamma"]), f["gamma"])
    assert rel_err(f32(L.Y), f["Y"]) <= TOL_BF16
    L.norm_eps = 0.0
    with pytest.raises(pqb.PqError):
        L.decode()


def test_decode_agrees_with_training_forward():
    c = I.make_linear_case(16, 512, 768, 64, 4, seed=5, exact_quota=False, with_grad=False)
    Ld = run_decode(c)
    Lt = PQLinear(16, 512, 768, 64, 4).load_case(c)
    Lt.pack(); Lt.forward()
    torch.cuda.synchronize()
    assert rel_err(f32(Ld.Y), f32(Lt.Y)) <= TOL_BF16
    assert np.array_equal(Ld.decode_view()["expert"].cpu().numpy(), Lt.saved_view()["expert"].cpu().numpy())


def test_decode_is_deterministic_and_repeatable():
    c = I.make_linear_case(7, 640, 1280, 96, 8, seed=6, exact_quota=False, with_grad=False)
    L = run_decode(c)
    y = L.Y.clone()
    for _ in range(3):
        L.decode()
    torch.cuda.synchronize()
    check_status()
    assert torch.equal(y, L.Y)


def test_decode_in_a_cuda_graph_and_without_dependent_launch():
    # Launches of different shapes (hence different shared-memory sizes) recorded in one CUDA graph replay to the
    # same bits as the eager calls, also after a later, smaller call; and the plain-launch option gives the same.
    shapes = [dict(T=2, K=2048, N=4096, r=64, E=4), dict(T=1, K=256, N=96, r=32, E=4), dict(T=11, K=1024, N=2560, r=160, E=8)]
    layers = []
    for i, kw in enumerate(shapes):
        c = I.make_linear_case(kw["T"], kw["K"], kw["N"], kw["r"], kw["E"], seed=70 + i, exact_quota=False, with_grad=False)
        L = PQLinear(c["T"], c["K"], c["N"], c["r"], c["E"], training=False, dump_acc=True).load_case(c)
        L.pack(bits_only=True)
        layers.append(L)
    eager = []
    for L in layers:
        L.decode()
        torch.cuda.synchronize()
        eager.append(L.Y.clone())
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            for L in layers:
                L.decode()
    layers[1].decode()                               # a small call after the capture
    torch.cuda.synchronize()
    for L in layers:
        L.Y.zero_()
    for _ in range(2):
        graph.replay()
    torch.cuda.synchronize()
    check_status()
    for L, y in zip(layers, eager):
        assert torch.equal(L.Y, y)
    pqb.pq_set_option(pqb.PQ_OPT_DECODE_PDL, 0)
    try:
        for L, y in zip(layers, eager):
            L.Y.zero_()
            L.decode()
            torch.cuda.synchronize()
            assert torch.equal(L.Y, y)
    finally:
        pqb.pq_set_option(pqb.PQ_OPT_DECODE_PDL, 1)
    check_status()


def test_decode_batch_of_independent_linears():
    # a mixed batch (different shapes, token counts, expert counts; more than one launch group of 16)
    # gives exactly what the separate calls give, and matches the oracle
    shapes = [dict(T=1, K=256, N=96, r=32, E=4), dict(T=16, K=512, N=2048, r=64, E=8), dict(T=5, K=2080, N=992, r=40, E=3),
              dict(T=3, K=1024, N=64, r=0, E=0), dict(T=9, K=384, N=320, r=160, E=1)]
    layers, cases = [], []
    for i in range(19):
        kw = dict(shapes[i % len(shapes)])
        c = I.make_linear_case(kw["T"], kw["K"], kw["N"], kw["r"], kw["E"], seed=40 + i, exact_quota=False, with_grad=False)
        L = PQLinear(c["T"], c["K"], c["N"], c["r"], c["E"], training=False, dump_acc=True).load_case(c)
        L.pack(bits_only=True)
        layers.append(L)
        cases.append(c)
    singles = []
    for L in layers:
        L.decode()
        torch.cuda.synchronize()
        singles.append(L.Y.clone())
        L.Y.zero_()
    items = pqb.make_decode_items([L.decode_entry() for L in layers])
    pqb.pq_decode_batch(items)
    torch.cuda.synchronize()
    check_status()
    for L, y, c in zip(layers, singles, cases):
        assert torch.equal(L.Y, y)
    for L, c in list(zip(layers, cases))[:5]:
        check_decode(c, L)


def test_decode_rejects_too_many_tokens():
    L = PQLinear(32, 256, 256, 32, 2, training=False)
    c = I.make_linear_case(32, 256, 256, 32, 2, seed=1, with_grad=False)
    L.load_case(c)
    L.pack(bits_only=True)
    assert pqb.pq_workspace_bytes(L.desc, pqb.PQ_PHASE_DECODE) == 0
    ws = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    with pytest.raises(pqb.PqError) as ei:
        pqb.pq_linear_forward(L.desc, L.X, L.w_bits, None, L.w_scales, L.A, L.B, L.Wr, L.alpha, L.beta, L.Y, None, ws)
    assert ei.value.status == pqb.PQ_ERR_SHAPE


@pytest.mark.parametrize("shape", [dict(T=1, K=256, N=96, r=32, E=4), dict(T=16, K=512, N=2048, r=64, E=8), dict(T=9, K=384, N=320, r=160, E=1),
                                   dict(T=5, K=2080, N=992, r=48, E=3), dict(T=2, K=512, N=288, r=256, E=2), dict(T=1, K=3200, N=8640, r=160, E=8),
                                   dict(T=4, K=8640, N=3200, r=160, E=8)])
def test_decode_int8_hp_branch_matches_oracle(shape):
    # Sec. 3.2 on the decode path: the branch multiplies the token's int8 codes by int8 expert matrices; every integer it
    # goes through (h_int, and with it the codes of h; z_int) must equal the oracle's, Y within the float tolerance.
    c = I.make_linear_case(shape["T"], shape["K"], shape["N"], shape["r"], shape["E"], seed=41)
    L = PQLinear(c["T"], c["K"], c["N"], c["r"], c["E"], training=False, dump_acc=True, guard=True).load_case(c)
    L.pack(bits_only=True)
    if L.w_bits_il is None:
        L.pack_decode()                  # the INT8 branch lives on the streaming kernel whatever the test's kernel choice
    L.pack_decode_hp8()
    L.decode()
    torch.cuda.synchronize()
    check_status()
    assert L.check_guards() == 0
    A8, gA, B8, gB = O.quantize_experts(c["A"], c["B"])
    assert np.array_equal(L.A8.cpu().numpy(), A8) and np.array_equal(L.B8.cpu().numpy(), B8)
    mu, lam = O.weight_scales(c["W"])
    bits = O.pack_bits(O.binarize(c["W"], mu))
    f = O.decode_forward(c["X"], bits, lam, c["A"], c["B"], c["Wr"], c["alpha"], c["beta"], hp_int8=(A8, gA, B8, gB))
    v = L.decode_view()
    assert np.array_equal(v["expert"].cpu().numpy(), f["idx"])
    assert np.array_equal(f32(v["gamma"]), f["gamma"])
    assert np.array_equal(v["acc"].cpu().numpy().astype(np.int64), f["acc"])
    assert np.array_equal(v["hp_h_int"].cpu().numpy().astype(np.int64), f["h_int"])
    assert np.array_equal(v["hp_z_int"].cpu().numpy().astype(np.int64), f["z_int"])
    assert rel_err(f32(L.Y), f["Y"]) <= TOL_BF16
    # and it is the INT8 branch, not the bf16 one
    fb = O.decode_forward(c["X"], bits, lam, c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
    assert not np.array_equal(fb["Y"], f["Y"])


def test_decode_int8_hp_branch_argument_errors():
    c = I.make_linear_case(2, 256, 128, 24, 2, seed=1)                   # r not a multiple of 16
    L = PQLinear(2, 256, 128, 24, 2, training=False).load_case(c)
    assert pqb.pq_decode_pack_hp8_bytes(L.desc) == 0
    c = I.make_linear_case(2, 256, 128, 32, 2, seed=1)
    L = PQLinear(2, 256, 128, 32, 2, training=False).load_case(c)
    L.pack(bits_only=True)
    if L.w_bits_il is None:
        L.pack_decode()
    L.pack_decode_hp8()
    entry = list(L.decode_entry())
    entry[13] = None                                                     # no streaming layout of the sign bits
    with pytest.raises(pqb.PqError) as ei:
        pqb.pq_decode_batch(pqb.make_decode_items([tuple(entry)]))
    assert ei.value.status == pqb.PQ_ERR_NULL


def test_decode_on_two_streams_at_once():
    # calls on different streams may overlap on the device: each stream's launches of the streaming kernel keep grid-barrier
    # words of their own, and every layer has its own workspace
    layers = []
    for i, kw in enumerate([dict(T=3, K=1024, N=2560, r=64, E=4), dict(T=1, K=2048, N=1024, r=32, E=8)]):
        c = I.make_linear_case(kw["T"], kw["K"], kw["N"], kw["r"], kw["E"], seed=90 + i, exact_quota=False, with_grad=False)
        L = PQLinear(c["T"], c["K"], c["N"], c["r"], c["E"], training=False, dump_acc=True).load_case(c)
        L.pack(bits_only=True)
        L.decode()
        layers.append(L)
    torch.cuda.synchronize()
    want = [L.Y.clone() for L in layers]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    for L in layers:
        L.Y.zero_()
    torch.cuda.synchronize()
    for _ in range(6):
        for L, s in zip(layers, streams):
            with torch.cuda.stream(s):
                L.decode()
    torch.cuda.synchronize()
    check_status()
    for L, y in zip(layers, want):
        assert torch.equal(L.Y, y)


def test_decode_batch_mixing_items_with_and_without_the_streaming_layout(decode_kernels):
    # a batch whose items only partly carry the streaming kernel's weight layout is cut into runs: the runs that carry it
    # go to the streaming kernel, the others to the two-kernel path; every item gets what a call of its own gives
    if decode_kernels == "pair":
        pytest.skip("needs the streaming layout")
    shapes = [dict(T=2, K=512, N=640, r=32, E=4), dict(T=1, K=1024, N=256, r=64, E=2), dict(T=7, K=256, N=1152, r=16, E=8)]
    layers = []
    for i in range(9):
        kw = shapes[i % 3]
        c = I.make_linear_case(kw["T"], kw["K"], kw["N"], kw["r"], kw["E"], seed=120 + i, exact_quota=False, with_grad=False)
        L = PQLinear(c["T"], c["K"], c["N"], c["r"], c["E"], training=False, dump_acc=True).load_case(c)
        L.pack(bits_only=True)
        L.decode()
        layers.append(L)
    torch.cuda.synchronize()
    want = [L.Y.clone() for L in layers]
    entries = []
    for i, L in enumerate(layers):
        e = list(L.decode_entry())
        if i in (2, 3, 7):          # these go without the layout
            e[13] = e[14] = None
        entries.append(tuple(e))
        L.Y.zero_()
    pqb.pq_decode_batch(pqb.make_decode_items(entries))
    torch.cuda.synchronize()
    check_status()
    for L, y in zip(layers, want):
        assert rel_err(f32(L.Y), f32(y)) <= 1e-2      # the two paths sum the expert product in different orders
    for i in (0, 1, 4, 5, 6, 8):
        assert torch.equal(layers[i].Y, want[i])


def test_decode_batch_items_that_share_their_activations(decode_kernels):
    # gate and up of a block (or q / k / v) read the same X: in one batch the streaming kernel quantises it once and the
    # later items multiply the first one's codes (App. A, no redundant reads).  Every item still gets exactly what a call
    # of its own gives, and its record (gamma, code sum) in its own workspace.
    shapes = [dict(T=3, K=1024, N=2560, r=64, E=4), dict(T=3, K=1024, N=640, r=32, E=8), dict(T=3, K=1024, N=1152, r=0, E=0)]
    layers, cases = [], []
    for i, kw in enumerate(shapes):
        c = I.make_linear_case(kw["T"], kw["K"], kw["N"], kw["r"], kw["E"], seed=140 + i, exact_quota=False, with_grad=False)
        L = PQLinear(c["T"], c["K"], c["N"], c["r"], c["E"], training=False, dump_acc=True).load_case(c)
        if i > 0:
            L.X = layers[0].X                     # the same tensor, not a copy
            c["X"] = cases[0]["X"]
        L.pack(bits_only=True)
        L.decode()
        layers.append(L)
        cases.append(c)
    torch.cuda.synchronize()
    want = [L.Y.clone() for L in layers]
    for L in layers:
        L.Y.zero_()
        L.ws_decode.zero_()
    pqb.pq_decode_batch(pqb.make_decode_items([L.decode_entry() for L in layers]))
    torch.cuda.synchronize()
    check_status()
    for L, y, c in zip(layers, want, cases):
        assert torch.equal(L.Y, y)
        check_decode(c, L)
