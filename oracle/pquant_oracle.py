"""CPU oracle for the pQuant decoupled linear layer.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition of what
the layer computes, written from the paper's equations.  It shares no code
with the CUDA path and must never be imported by the product package; only
the tests, the smoke check and the benchmark's CPU-baseline leg call it.

Everything is numpy.  Sums run in fp64 (a BLAS matmul serves as the "sum
over k" step); integer results are exact; bf16 tensors are passed in as
float32/float64 arrays whose values are bf16-representable.

Notation (paper, Sec. 3):  X[T,K] activations (one row per token), latent
W[N,K] (the paper's W in R^{m x n}, Y = W X per token), mu / lam the
weight mean / mean-absolute value (Eq. 6), gamma_t the per-token activation
scale (Eq. 9), alpha / beta the feature scales of the high-precision (HP) and
1-bit branches (Eq. 11), A_e[r,K], B_e[N,r] the two factors of HP expert e,
Wr[E,K] the router (Sec. 3.3).

Readings taken where the paper is silent or garbled (each is listed again in
the design notes of the repository):
  * Sign(0) := +1, i.e. the bit is  W >= mu  (Eq. 4 leaves 0 undefined).
  * lam is the mean |W| of the *uncentred* W (Eq. 6, literal).
  * activations: one gamma per token row; gamma = 128 / max(amax, 1e-5);
    round half to even; int8 result clipped to [-128, 127] (Eq. 7-9; the
    printed clip bounds with epsilon are subsumed by the integer clamp).
  * router: no bias, softmax over the E logits, top-1, lowest index wins
    ties, the branch output is multiplied by the selected probability.
  * HP branch: bf16 weights on the un-quantised bf16 input, no
    non-linearity between the two factors.
  * STE (App. B.1): Sign, Round and Clip have derivative 1; mu, lam and
    gamma are constants for the backward pass; dW uses the de-quantised
    activations q/gamma that the forward really multiplied.

parity unpinned: absolute output values on random inputs (the paper prints no
worked example); every function below is pinned instead by invariants, closed
forms, brute force and finite differences in tests/test_oracle_*.py.
"""
from __future__ import annotations

import numpy as np

ACT_QMAX = np.float32(128.0)      # 2^7 in Eq. 9
ACT_AMAX_FLOOR = np.float32(1e-5)  # guards the all-zero row (paper silent)


# --------------------------------------------------------------------------
# small numeric helpers
# --------------------------------------------------------------------------
def round_to_bf16(x):
    """Round fp64 values once to the nearest bf16 value (ties to even).

    bf16 keeps 8 significand bits: write x = m * 2^e with m in [0.5, 1) and
    round m to a multiple of 2^-8.  Normal range only (tests stay inside it).
    """
    x = np.asarray(x, dtype=np.float64)
    m, e = np.frexp(x)
    return np.ldexp(np.rint(m * 256.0) / 256.0, e)


# --------------------------------------------------------------------------
# 1-bit branch: weights (Eq. 3, 4, 6; packing App. A)
# --------------------------------------------------------------------------
def weight_scales(W):
    """Eq. 6: mu = mean(W), lam = mean(|W|) over the whole matrix.

    fp64 sums, each rounded once to fp32 (mu decides sign bits, so its
    precision is part of the definition the GPU must reproduce).
    """
    W64 = np.asarray(W, dtype=np.float64)
    n = W64.size
    mu = np.float32(W64.sum() / n)
    lam = np.float32(np.abs(W64).sum() / n)
    return mu, lam


def binarize(W, mu):
    """Eq. 3-4: S = Sign(W - mu) in {+1, -1}, with Sign(0) := +1.

    Decided as the fp32 comparison W >= mu (no subtraction, so no rounding).
    """
    W32 = np.asarray(W, dtype=np.float32)
    return np.where(W32 >= np.float32(mu), 1, -1).astype(np.int8)


def pack_bits(S):
    """App. A: 1-bit storage.  Bit j of word i of a row holds k = 32 i + j,
    bit value 1 <-> +1.  Read as bytes (little endian) this is the paper's
    "8 parameters per uint8" stream, LSB first."""
    S = np.asarray(S)
    N, K = S.shape
    assert K % 32 == 0
    b = (S > 0).astype(np.uint64).reshape(N, K // 32, 32)
    weights = (np.uint64(1) << np.arange(32, dtype=np.uint64))
    return (b * weights).sum(axis=2).astype(np.uint32)


def unpack_bits(bits, K):
    """Inverse of pack_bits: uint32 words -> S in {+1,-1} int8 [N,K]."""
    bits = np.asarray(bits, dtype=np.uint32)
    N = bits.shape[0]
    j = np.arange(32, dtype=np.uint32)
    b = (bits[:, :, None] >> j) & np.uint32(1)
    return (2 * b.astype(np.int8) - 1).reshape(N, K)


# --------------------------------------------------------------------------
# 1-bit branch: activations (Eq. 7-9) and the W1A8 product (Eq. 10)
# --------------------------------------------------------------------------
def act_quant(X):
    """Eq. 7-9 per token row: gamma = 2^7 / max|x|, q = RoundClip(x*gamma).

    All in fp32 exactly as written: one IEEE division, one IEEE multiply per
    element, round half to even, clamp to the int8 range [-128, 127].
    Returns q int8 [T,K], gamma fp32 [T].
    """
    X32 = np.asarray(X, dtype=np.float32)
    amax = np.max(np.abs(X32), axis=1) if X32.shape[1] else np.zeros(X32.shape[0], np.float32)
    amax = np.maximum(amax.astype(np.float32), ACT_AMAX_FLOOR)
    gamma = (ACT_QMAX / amax).astype(np.float32)
    scaled = (X32 * gamma[:, None]).astype(np.float32)
    q = np.clip(np.rint(scaled), -128.0, 127.0).astype(np.int8)
    return q, gamma


def onebit_gemm(q, S):
    """Eq. 10, integer part: acc[t,n] = sum_k q[t,k] * S[n,k], exact.

    The fp64 matmul is exact here: |acc| <= 128 K << 2^53.
    """
    acc = np.asarray(q, dtype=np.float64) @ np.asarray(S, dtype=np.float64).T
    acc = np.rint(acc).astype(np.int64)
    assert np.all(np.abs(acc) < 2 ** 31)
    return acc


def onebit_dequant(acc, lam, gamma):
    """Eq. 10: y1 = (lam / gamma_t) * acc, fp64."""
    return acc.astype(np.float64) * (np.float64(lam) / gamma.astype(np.float64))[:, None]


# --------------------------------------------------------------------------
# router (Sec. 3.3) and permutation
# --------------------------------------------------------------------------
def router_logits_fp32(X, Wr):
    """Router logits in the fp32 summation order that decides the top-1 index.

    The decision is an integer, so both implementations must take it in the
    same arithmetic: fp32, products of two bf16 values (exact in fp32), 32
    interleaved partial sums where partial j takes the 8-element chunks c with
    c mod 32 == j in ascending k (fused multiply-add), combined by the
    butterfly tree with lane distances 16, 8, 4, 2, 1.  Because each product
    is exact, fl32(sum + product) equals the fused multiply-add.
    """
    X32 = np.asarray(X, dtype=np.float32)
    W32 = np.asarray(Wr, dtype=np.float32)
    T, K = X32.shape
    E = W32.shape[0]
    assert K % 8 == 0
    part = np.zeros((T, E, 32), dtype=np.float32)
    for c in range(K // 8):
        j = c % 32
        for i in range(8):
            k = 8 * c + i
            prod = (X32[:, k:k + 1] * W32[None, :, k]).astype(np.float32)  # exact
            part[:, :, j] = (part[:, :, j] + prod).astype(np.float32)
    for d in (16, 8, 4, 2, 1):
        idx = np.arange(32) ^ d
        part = (part + part[:, :, idx]).astype(np.float32)
    return part[:, :, 0]


def router(X, Wr, top_k=1):
    """Sec. 3.3: one linear layer, softmax gate, top-1 (lowest index on ties).

    Returns dict: logits32 (decision arithmetic), logits64, probs (fp64
    softmax of logits32), idx int32 [T], gate fp64 [T] = probs[idx], margin
    (fp64 top-1 minus top-2 logit).
    With Wr None (E <= 1): idx = 0, gate = 1, no router.
    """
    X64 = np.asarray(X, dtype=np.float64)
    T = X64.shape[0]
    if Wr is None:
        return dict(logits32=None, logits64=None, probs=np.ones((T, 1)), idx=np.zeros(T, np.int32),
                    gate=np.ones(T), margin=np.full(T, np.inf))
    l32 = router_logits_fp32(X, Wr)
    l64 = X64 @ np.asarray(Wr, dtype=np.float64).T
    z = l32.astype(np.float64)
    z = z - z.max(axis=1, keepdims=True)
    p = np.exp(z)
    p /= p.sum(axis=1, keepdims=True)
    idx = np.argmax(l32, axis=1).astype(np.int32)          # first maximum = lowest index
    gate = p[np.arange(T), idx]
    srt = np.sort(l64, axis=1)
    margin = srt[:, -1] - srt[:, -2] if l64.shape[1] > 1 else np.full(T, np.inf)
    return dict(logits32=l32, logits64=l64, probs=p, idx=idx, gate=gate, margin=margin)


def permutation(idx, E):
    """Token permutation implied by sparse activation: histogram over experts,
    exclusive scan, stable scatter.  perm[p] = token at sorted position p,
    offsets[e] .. offsets[e+1] = positions of expert e."""
    idx = np.asarray(idx)
    counts = np.bincount(idx, minlength=E)
    offsets = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    perm = np.argsort(idx, kind="stable").astype(np.int32)
    return perm, offsets


# --------------------------------------------------------------------------
# high-precision branch (Sec. 3.2, 3.3)
# --------------------------------------------------------------------------
def hp_branch(X, A, B, idx):
    """h_t = A_e x_t, z_t = B_e h_t for the token's expert e = idx[t]; fp64,
    h is not rounded.  A [E,r,K], B [E,N,r]."""
    X64 = np.asarray(X, dtype=np.float64)
    A64 = np.asarray(A, dtype=np.float64)
    B64 = np.asarray(B, dtype=np.float64)
    T = X64.shape[0]
    E, r, _ = A64.shape
    N = B64.shape[1]
    h = np.zeros((T, r))
    z = np.zeros((T, N))
    for e in range(E):
        sel = np.nonzero(idx == e)[0]
        if sel.size:
            h[sel] = X64[sel] @ A64[e].T
            z[sel] = h[sel] @ B64[e].T
    return h, z


def hp_branch_all_experts(X, A, B, weights):
    """Every expert active (top_k = E): z_t = sum_e weights[t,e] * B_e A_e x_t.
    Used only to check that the routed form reduces to the dense one."""
    X64 = np.asarray(X, dtype=np.float64)
    E = A.shape[0]
    z = 0.0
    for e in range(E):
        h = X64 @ np.asarray(A[e], dtype=np.float64).T
        z = z + weights[:, e:e + 1] * (h @ np.asarray(B[e], dtype=np.float64).T)
    return z


# --------------------------------------------------------------------------
# high-precision branch in INT8 (Sec. 3.2: the branch runs at 8-bit precision,
# its weights quantised the way the 8-bit activations are)
# --------------------------------------------------------------------------
def absmax_quant_matrix(Wm):
    """Eq. 7-9 applied to a whole weight matrix: gamma_W = 2^7 / max|W| (one scale
    per matrix, as the 1-bit branch has one lam per matrix), W8 = RoundClip(W * gamma_W)
    in [-128, 127].  Same fp32 arithmetic as act_quant.  Returns W8 int8, gamma_W fp32."""
    W32 = np.asarray(Wm, dtype=np.float32)
    amax = np.maximum(np.float32(np.max(np.abs(W32))) if W32.size else np.float32(0), ACT_AMAX_FLOOR)
    gamma = np.float32(ACT_QMAX / amax)
    q = np.clip(np.rint((W32 * gamma).astype(np.float32)), -128.0, 127.0).astype(np.int8)
    return q, gamma


def quantize_experts(A, B):
    """absmax_quant_matrix for every expert's two matrices: A8 [E,r,K], gA [E], B8 [E,N,r], gB [E]."""
    E = A.shape[0]
    A8, B8 = np.zeros(A.shape, np.int8), np.zeros(B.shape, np.int8)
    gA, gB = np.zeros(E, np.float32), np.zeros(E, np.float32)
    for e in range(E):
        A8[e], gA[e] = absmax_quant_matrix(A[e])
        B8[e], gB[e] = absmax_quant_matrix(B[e])
    return A8, gA, B8, gB


def requant_hidden(h_int):
    """The hidden activation of the INT8 branch is an exact integer, h_int = A8 q; it enters the second 8-bit linear
    quantised per token like any activation (Eq. 7-9).  Its real value is h_int / (gamma_A gamma_t), a positive
    multiple of the integer, so the codes can be taken from the integers themselves:
        gamma_h = fl32(128 / max(fl32(max_j |h_int|), 1e-5)),  qh = RoundClip(fl32(fl32(h_int) * gamma_h)),
    every step one IEEE fp32 operation (the conversion of an integer above 2^24 rounds to nearest even).
    Returns qh int8 [T,r], gamma_h fp32 [T] (the scale relative to h_int)."""
    h32 = np.asarray(h_int, dtype=np.int64).astype(np.float32)
    amax = np.max(np.abs(h32), axis=1) if h32.shape[1] else np.zeros(h32.shape[0], np.float32)
    gamma_h = (ACT_QMAX / np.maximum(amax.astype(np.float32), ACT_AMAX_FLOOR)).astype(np.float32)
    qh = np.clip(np.rint((h32 * gamma_h[:, None]).astype(np.float32)), -128.0, 127.0).astype(np.int8)
    return qh, gamma_h


def hp_branch_int8(q, gamma, A8, gA, B8, gB, idx):
    """INT8 high-precision branch on the int8 activation codes q (the same codes the 1-bit branch multiplies):
        h_int = A8_e q_t   (exact)        ->  qh, gamma_h = requant_hidden(h_int)
        z_int = B8_e qh_t  (exact)        ->  z = z_int / (gamma_B gamma_h gamma_A gamma_t)   (fp64)
    Returns dict(h_int, qh, gamma_h, z_int, z, scale) with scale[t] the fp64 factor z / z_int."""
    q64 = np.asarray(q, dtype=np.int64)
    T = q64.shape[0]
    E, r, _ = A8.shape
    N = B8.shape[1]
    h_int = np.zeros((T, r), np.int64)
    for e in range(E):
        sel = np.nonzero(idx == e)[0]
        if sel.size:
            h_int[sel] = q64[sel] @ A8[e].astype(np.int64).T
    assert np.all(np.abs(h_int) < 2 ** 31)
    qh, gamma_h = requant_hidden(h_int)
    z_int = np.zeros((T, N), np.int64)
    for e in range(E):
        sel = np.nonzero(idx == e)[0]
        if sel.size:
            z_int[sel] = qh[sel].astype(np.int64) @ B8[e].astype(np.int64).T
    scale = 1.0 / (gB.astype(np.float64)[idx] * gamma_h.astype(np.float64) * gA.astype(np.float64)[idx] * np.asarray(gamma, np.float64))
    return dict(h_int=h_int, qh=qh, gamma_h=gamma_h, z_int=z_int, z=z_int * scale[:, None], scale=scale)


# --------------------------------------------------------------------------
# the layer: forward (Eq. 10 + Eq. 11) and STE backward (App. B.1)
# --------------------------------------------------------------------------
def _scale_vec(s, N):
    s = np.asarray(s, dtype=np.float64).reshape(-1)
    assert s.size in (1, N)
    return np.broadcast_to(s, (N,)) if s.size == 1 else s


def linear_forward(X, W, A=None, B=None, Wr=None, alpha=1.0, beta=1.0, S=None, lam=None, hp_int8=None):
    """Forward of the decoupled linear layer.

    Y[t,n] = alpha_n * g_t * z_t[n] + beta_n * (lam/gamma_t) * acc[t,n]   (Eq. 10, 11)
    rounded once to bf16.  A/B None -> pure 1-bit layer (the MHA form).
    S/lam may be given instead of W (decode path from stored bits).
    hp_int8: None -> bf16 HP branch on the un-quantised input; True -> the paper's INT8 branch, A and B
    quantised here (quantize_experts); a tuple (A8, gA, B8, gB) -> the INT8 branch on stored int8 experts.
    Returns a dict with every intermediate.
    """
    out = {}
    if S is None:
        mu, lam = weight_scales(W)
        S = binarize(W, mu)
        out["mu"] = mu
    N = S.shape[0]
    out["lam"], out["S"] = lam, S
    q, gamma = act_quant(X)
    acc = onebit_gemm(q, S)
    y1 = onebit_dequant(acc, lam, gamma)
    out.update(q=q, gamma=gamma, acc=acc, y1=y1)
    al, be = _scale_vec(alpha, N), _scale_vec(beta, N)
    T = np.asarray(X).shape[0]
    if A is not None and A.shape[1] > 0:
        E = A.shape[0]
        rt = router(X, Wr if E > 1 else None)
        if hp_int8 is None:
            h, z = hp_branch(X, A, B, rt["idx"])
        else:
            A8, gA, B8, gB = quantize_experts(A, B) if hp_int8 is True else hp_int8
            hp = hp_branch_int8(q, gamma, A8, gA, B8, gB, rt["idx"])
            h, z = hp["h_int"] / (gA.astype(np.float64)[rt["idx"]] * gamma.astype(np.float64))[:, None], hp["z"]
            out.update(A8=A8, gA=gA, B8=B8, gB=gB, h_int=hp["h_int"], qh=hp["qh"], gamma_h=hp["gamma_h"], z_int=hp["z_int"])
        perm, offsets = permutation(rt["idx"], E)
        out.update(h=h, z=z, perm=perm, offsets=offsets, **rt)
        y64 = al[None, :] * rt["gate"][:, None] * z + be[None, :] * y1
    else:
        out.update(idx=np.zeros(T, np.int32), gate=np.ones(T), z=np.zeros((T, N)))
        y64 = be[None, :] * y1
    out["Y64"] = y64
    out["Y"] = round_to_bf16(y64)
    return out


def linear_backward(dY, X, fwd, A=None, B=None, Wr=None, alpha=1.0, beta=1.0):
    """Straight-through backward of linear_forward (App. B.1).

    fwd is the dict linear_forward returned.  Gradients (fp64; dX also given
    rounded to bf16):
      D1 = beta*dY;  dX1 = lam * D1 S;  dW = D1^T (q/gamma);  dbeta_n = sum_t dY*y1
      O = alpha*dY;  dalpha_n = sum_t dY*g*z;  dg_t = sum_n O*z;  dZ = g*O
      dB_e = sum_{t in e} dZ_t h_t^T;  dH = dZ B_e;  dA_e = sum dH_t x_t^T;  dX2 = dH A_e
      dl[t,j] = dg_t g_t (delta_{j,e} - p[t,j]);  dWr = dl^T X;  dX3 = dl Wr
    dalpha/dbeta are returned per output feature [N]; their sum is the
    gradient of a scalar feature scale.
    """
    dY64 = np.asarray(dY, dtype=np.float64)
    X64 = np.asarray(X, dtype=np.float64)
    S64 = fwd["S"].astype(np.float64)
    N = S64.shape[0]
    T = X64.shape[0]
    lam = np.float64(fwd["lam"])
    al, be = _scale_vec(alpha, N), _scale_vec(beta, N)
    g = {}
    D1 = dY64 * be[None, :]
    xt = fwd["q"].astype(np.float64) / fwd["gamma"].astype(np.float64)[:, None]
    dX = lam * (D1 @ S64)
    g["dX1"] = dX.copy()
    g["dW"] = D1.T @ xt
    g["dbeta"] = (dY64 * fwd["y1"]).sum(axis=0)
    if A is not None and A.shape[1] > 0:
        A64 = np.asarray(A, dtype=np.float64)
        B64 = np.asarray(B, dtype=np.float64)
        E = A64.shape[0]
        idx, gate, z, h = fwd["idx"], fwd["gate"], fwd["z"], fwd["h"]
        O = dY64 * al[None, :]
        g["dalpha"] = (dY64 * gate[:, None] * z).sum(axis=0)
        dg = (O * z).sum(axis=1)
        dZ = gate[:, None] * O
        dA = np.zeros_like(A64)
        dB = np.zeros_like(B64)
        dX2 = np.zeros_like(X64)
        for e in range(E):
            sel = np.nonzero(idx == e)[0]
            if sel.size == 0:
                continue
            dB[e] = dZ[sel].T @ h[sel]
            dH = dZ[sel] @ B64[e]
            dA[e] = dH.T @ X64[sel]
            dX2[sel] = dH @ A64[e]
        g.update(dA=dA, dB=dB, dg=dg)
        dX = dX + dX2
        if E > 1:
            Wr64 = np.asarray(Wr, dtype=np.float64)
            p = fwd["probs"]
            onehot = np.zeros((T, E))
            onehot[np.arange(T), idx] = 1.0
            dl = (dg * gate)[:, None] * (onehot - p)
            g["dWr"] = dl.T @ X64
            g["dl"] = dl
            dX = dX + dl @ Wr64
    else:
        g["dalpha"] = np.zeros(N)
    g["dX64"] = dX
    g["dX"] = round_to_bf16(dX)
    return g


# --------------------------------------------------------------------------
# FFN-level decoupling (Eq. 11, Table 1): two parallel FFNs split along the hidden dimension
# --------------------------------------------------------------------------
def silu_fp32(g32):
    """SiLU in the arithmetic both sides can reproduce: the logistic factor in fp64, rounded once to fp32, then one
    fp32 multiply.  (An fp32 exponential differs from library to library in its last bit, and the result feeds a
    quantiser.)"""
    g32 = np.asarray(g32, dtype=np.float32)
    s32 = (1.0 / (1.0 + np.exp(-g32.astype(np.float64)))).astype(np.float32)
    return (g32 * s32).astype(np.float32)


def ffn_int8(q, gamma, G8, gG, U8, gU, D8, gD):
    """The INT8 FFN of hidden width r on the int8 activation codes q (Sec. 3.2, Eq. 11 first term; the LLaMA-style
    gated form the paper's models use):
        g = (G8 q) / (gamma_G gamma_t),  u = (U8 q) / (gamma_U gamma_t)       exact integers, de-quantised in fp32
        m = silu(g) * u                                                       fp32
        qm, gamma_m = Eq. 7-9 on m (per token)
        z = (D8 qm) / (gamma_D gamma_m)
    Every step up to the codes qm is pinned fp32 arithmetic: deq = fl(1 / fl(gamma_W gamma_t)), g = fl(fl(g_int) deq),
    m = fl(silu_fp32(g) u).  Returns dict(g_int, u_int, m, qm, gamma_m, z_int, z)."""
    q64 = np.asarray(q, dtype=np.int64)
    g_int = q64 @ G8.astype(np.int64).T
    u_int = q64 @ U8.astype(np.int64).T
    assert np.all(np.abs(g_int) < 2 ** 31) and np.all(np.abs(u_int) < 2 ** 31)
    gamma = np.asarray(gamma, dtype=np.float32)
    deq_g = (np.float32(1.0) / (np.float32(gG) * gamma).astype(np.float32)).astype(np.float32)
    deq_u = (np.float32(1.0) / (np.float32(gU) * gamma).astype(np.float32)).astype(np.float32)
    g32 = (g_int.astype(np.float32) * deq_g[:, None]).astype(np.float32)
    u32 = (u_int.astype(np.float32) * deq_u[:, None]).astype(np.float32)
    m32 = (silu_fp32(g32) * u32).astype(np.float32)
    qm, gamma_m = act_quant(m32)
    z_int = qm.astype(np.int64) @ D8.astype(np.int64).T
    z = z_int / (np.float64(gD) * gamma_m.astype(np.float64))[:, None]
    return dict(g_int=g_int, u_int=u_int, m=m32, qm=qm, gamma_m=gamma_m, z_int=z_int, z=z)


def ffn_decoupled_forward(X, Wg, Wu, Wd, G, U, D, alpha=2.0, beta=0.2):
    """Eq. 11: Y = alpha FFN_INT8[:r](x) + beta FFN_INT1[r:](x), both FFNs gated (down(silu(gate x) * up x)).
    Wg, Wu [F1, Dm], Wd [Dm, F1]: latent weights of the 1-bit FFN of hidden width F1 = D_ff - r, each a pure 1-bit
    linear (Eq. 3-10) whose output is a bf16 tensor; G, U [r, Dm], D [Dm, r]: the INT8 FFN's matrices (bf16 values),
    quantised per matrix.  The 1-bit FFN's hidden activation is bf16(silu(g1) * u1) with the product taken in fp64.
    Returns dict with the pieces; Y rounded once to bf16."""
    fg = linear_forward(X, Wg, beta=1.0)
    fu = linear_forward(X, Wu, beta=1.0)
    g1, u1 = fg["Y"], fu["Y"]
    m1 = round_to_bf16(g1 / (1.0 + np.exp(-g1)) * u1)
    fd = linear_forward(m1, Wd, beta=1.0)
    G8, gG = absmax_quant_matrix(G)
    U8, gU = absmax_quant_matrix(U)
    D8, gD = absmax_quant_matrix(D)
    hp = ffn_int8(fg["q"], fg["gamma"], G8, gG, U8, gU, D8, gD)
    y64 = np.float64(alpha) * hp["z"] + np.float64(beta) * fd["y1"]
    return dict(gate=fg, up=fu, down=fd, m1=m1, hp=hp, G8=G8, U8=U8, D8=D8, gG=gG, gU=gU, gD=gD, Y64=y64, Y=round_to_bf16(y64))


def rmsnorm(X, weight, eps):
    """RMSNorm in front of the activation quantiser (App. A: at inference the norm is
    fused with the quantisation; the equations write it as LayerNorm(X)).

    Per token row: x / sqrt(mean_k x^2 + eps) * weight.  The paper fixes no
    precision; the reading taken is: the mean of squares and the reciprocal
    square root in fp64, that factor rounded once to fp32, then two fp32
    multiplies per element (by the factor, then by the gain), and one rounding
    to bf16 -- the values a separate bf16 norm layer would have handed over.
    """
    X32 = np.asarray(X, dtype=np.float32)
    w32 = np.asarray(weight, dtype=np.float32)
    ms = np.mean(np.square(X32.astype(np.float64)), axis=1)
    rinv = (1.0 / np.sqrt(ms + np.float64(np.float32(eps)))).astype(np.float32)
    y = ((X32 * rinv[:, None]).astype(np.float32) * w32[None, :]).astype(np.float32)
    return round_to_bf16(y.astype(np.float64)).astype(np.float32)


def decode_forward(X, bits, lam, A=None, B=None, Wr=None, alpha=1.0, beta=1.0, norm_weight=None, norm_eps=1e-6, hp_int8=None):
    """Inference path (App. A): same forward, with S read back out of the
    packed 1-bit words instead of the latent weights; with `norm_weight` the
    input is the un-normalised activation and RMSNorm comes first."""
    if norm_weight is not None:
        X = rmsnorm(X, norm_weight, norm_eps)
    K = np.asarray(X).shape[1]
    return linear_forward(X, None, A, B, Wr, alpha, beta, S=unpack_bits(bits, K), lam=lam, hp_int8=hp_int8)
