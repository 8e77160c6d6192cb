"""GPU parity of the decoder harness: a small LLaMA-style decoder whose projections all go through the C ABI
(pack + forward in the forward pass, backward in the backward pass, via torch.autograd).  The torch parts between
the projections are not under test; what is checked is that every projection, fed by and feeding foreign kernels,
still computes the layer: its captured input and upstream gradient are replayed through the CPU oracle."""
import math

import numpy as np
import pytest
import torch

from oracle import pquant_oracle as O
from paper_2602_22592_b200 import binding as pqb
from paper_2602_22592_b200.decoder_harness import PQDecoder
from test_gpu_forward import TOL_BF16, TOL_RMS, check_status, f32, rel_err, rms_err

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("attn_hp", [True, False])
def test_small_decoder_step_matches_oracle_per_projection(attn_hp):
    m = PQDecoder(layers=2, hidden=256, heads=4, ffn=512, vocab=1000, batch=2, seq=64, r=32, E=4, attn_hp=attn_hp, seed=5)
    for L in m.linears():
        L.capture = {}
    ids, tgt = m.random_batch()
    m.timer.enabled = True
    loss = m.step(ids, tgt)
    torch.cuda.synchronize()
    check_status()
    assert m.timer.total_ms() > 0
    assert abs(float(loss) - math.log(1000)) < 0.5          # random initialisation: near the uniform prediction
    assert m.embed.grad is not None and torch.isfinite(m.embed.grad.float()).all()
    n = 0
    for L in m.linears():
        cap = L.capture
        assert set(cap) == {"x", "y", "dy", "dx"}, L.name
        X, dY = f32(cap["x"]), f32(cap["dy"])
        A = None if L.A is None else f32(L.A)
        B = None if L.B is None else f32(L.B)
        Wr = None if L.Wr is None else f32(L.Wr)
        f = O.linear_forward(X, f32(L.W), A, B, Wr, f32(L.alpha), f32(L.beta))
        g = O.linear_backward(dY, X, f, A, B, Wr, f32(L.alpha), f32(L.beta))
        assert np.array_equal(L.w_s8.cpu().numpy(), f["S"]), L.name
        if L.r > 0:
            sv = pqb.pq_saved_view_init(L.desc, L.saved)
            assert np.array_equal(sv["expert"].cpu().numpy(), f["idx"]), L.name
        pairs = {"y": (f32(cap["y"]), f["Y"]), "dx": (f32(cap["dx"]), g["dX"]), "dW": (f32(L.dW), g["dW"])}
        if L.r > 0:
            pairs["dA"] = (f32(L.dA), g["dA"])
            pairs["dB"] = (f32(L.dB), g["dB"])
            pairs["dWr"] = (f32(L.dWr), g["dWr"])
        for k, (a, b) in pairs.items():
            assert rel_err(a, b) <= TOL_BF16, (L.name, k, rel_err(a, b))
            assert rms_err(a, b) <= TOL_RMS, (L.name, k, rms_err(a, b))
        n += 1
    assert n == 14
