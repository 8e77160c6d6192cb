"""Seeded synthetic inputs for the pQuant linear layer.

Serves the CUDA tests, the CPU oracle tests and the benchmark alike, and holds
none of the layer's arithmetic: only random draws shaped like the paper's
LLaMA-style workloads (Sec. 4.1, App. C: hidden 2048 / FFN 5632 at 1.3B;
N(0, 0.02) initialisation; sequence 2048) and rounding of those draws to the
storage type.  numpy only; no torch, no CUDA.

bf16 tensors are returned as float32 arrays whose values are exactly
bf16-representable, so `torch.from_numpy(a).to(torch.bfloat16)` is lossless
and the oracle can read the very same numbers.
"""
from __future__ import annotations

import numpy as np

# Zipf(1.1) token-to-expert skew over 8 experts: share_e proportional to e^-1.1
ZIPF_EXPONENT = 1.1


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed, stream]))


def bf16_values(x: np.ndarray) -> np.ndarray:
    """Round float32 to the nearest bf16 value (ties to even), returned as float32."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    u = (u + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    return u.view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of an array already holding bf16-representable float32 values."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    assert not np.any(u & np.uint32(0xFFFF)), "values are not bf16-representable"
    return (u >> np.uint32(16)).astype(np.uint16)


def zipf_shares(E: int, s: float = ZIPF_EXPONENT) -> np.ndarray:
    p = np.arange(1, E + 1, dtype=np.float64) ** (-s)
    return p / p.sum()


def zipf_assignment(T: int, E: int, rng: np.random.Generator, exact_quota: bool) -> np.ndarray:
    """Planted expert id per token.  exact_quota: expert e gets round(share_e*T)
    tokens (largest-remainder fix-up), shuffled; else i.i.d. draws (small T)."""
    p = zipf_shares(E)
    if not exact_quota:
        return rng.choice(E, size=T, p=p).astype(np.int32)
    quota = np.floor(p * T).astype(np.int64)
    rem = T - quota.sum()
    order = np.argsort(-(p * T - quota), kind="stable")
    quota[order[:rem]] += 1
    ids = np.repeat(np.arange(E, dtype=np.int32), quota)
    rng.shuffle(ids)
    return ids


def router_weights(E: int, K: int, rng: np.random.Generator, orthonormal: bool) -> np.ndarray:
    """Router rows: E orthonormal directions (planted routing) or N(0, 0.02)."""
    if orthonormal:
        g = rng.standard_normal((K, E))
        qm, _ = np.linalg.qr(g)
        return bf16_values(qm.T.astype(np.float32))
    return bf16_values((0.02 * rng.standard_normal((E, K))).astype(np.float32))


def make_linear_case(T: int, K: int, N: int, r: int, E: int, seed: int, *,
                     scale_vector: bool = False, alpha: float = 2.0, beta: float = 0.2,
                     zipf: bool = True, exact_quota: bool | None = None,
                     plant: float = 6.0, with_grad: bool = True) -> dict:
    """One pQuant linear: X, latent W, HP experts A/B, router Wr, feature scales, dY.

    Returns float32 arrays (bf16-valued where the layer stores bf16):
      X [T,K] ~ N(0,1) bf16;  W [N,K] ~ N(0, 0.02) fp32;
      A [E,r,K], B [E,N,r] ~ N(0, 0.02) bf16;  Wr [E,K] bf16 (E > 1);
      alpha, beta fp32 of length 1 (paper's scalars) or N (vector form);
      dY [T,N] ~ N(0,1) bf16.
    With E > 1 and zipf, a Zipf(1.1) assignment is planted by adding
    plant * Wr[e_t] to token t before rounding, so the router computes it.
    """
    case = dict(T=T, K=K, N=N, r=r, E=E, seed=seed)
    X = _rng(seed, 0).standard_normal((T, K), dtype=np.float32)
    case["W"] = (np.float32(0.02) * _rng(seed, 1).standard_normal((N, K), dtype=np.float32))
    if r > 0 and E > 0:
        case["A"] = bf16_values(np.float32(0.02) * _rng(seed, 2).standard_normal((E, r, K), dtype=np.float32))
        case["B"] = bf16_values(np.float32(0.02) * _rng(seed, 3).standard_normal((E, N, r), dtype=np.float32))
    else:
        case["A"] = case["B"] = None
    case["Wr"] = None
    if E > 1:
        rr = _rng(seed, 4)
        Wr = router_weights(E, K, rr, orthonormal=zipf)
        case["Wr"] = Wr
        if zipf:
            quota = exact_quota if exact_quota is not None else (T >= 64 * E)
            planted = zipf_assignment(T, E, rr, quota)
            X = X + np.float32(plant) * Wr[planted]
            case["planted"] = planted
    case["X"] = bf16_values(X)
    n_scale = N if scale_vector else 1
    case["alpha"] = np.full(n_scale, alpha, dtype=np.float32)
    case["beta"] = np.full(n_scale, beta, dtype=np.float32)
    if with_grad:
        case["dY"] = bf16_values(_rng(seed, 5).standard_normal((T, N), dtype=np.float32))
    return case


# The benchmark configurations (shapes of a 1.3B / 3B LLaMA-style model).
def config1() -> dict:
    """Small single layer: 256 tokens x 512 -> 512, one dense HP branch of width 32,
    feature-scale vectors of ones."""
    return make_linear_case(256, 512, 512, 32, 1, seed=0, scale_vector=True, alpha=1.0, beta=1.0)


MLP_1P3B = dict(T=8192, hidden=2048, ffn=5632, r=128)
DECODE_3B = dict(hidden=3200, ffn=8640, r=160, E=8)


def mlp_shapes(hidden: int, ffn: int) -> list[tuple[str, int, int]]:
    """(name, K, N) of the three MLP projections."""
    return [("gate", hidden, ffn), ("up", hidden, ffn), ("down", ffn, hidden)]


def config_mlp(E: int, seed: int, T: int | None = None) -> list[dict]:
    """1.3B-shaped MLP projections (gate/up/down) as independent pQuant linears.
    E = 1: dense HP branch (config 2);  E = 8: routed experts with Zipf skew (config 3)."""
    T = MLP_1P3B["T"] if T is None else T
    cases = []
    for i, (name, K, N) in enumerate(mlp_shapes(MLP_1P3B["hidden"], MLP_1P3B["ffn"])):
        c = make_linear_case(T, K, N, MLP_1P3B["r"], E, seed=seed * 16 + i)
        c["name"] = name
        cases.append(c)
    return cases


def config_decode(M: int, seed: int = 4, layers: int = 1) -> list[dict]:
    """3B-shaped decode linears: M tokens, packed 1-bit weights, 8 experts of width 160."""
    cases = []
    for layer in range(layers):
        for i, (name, K, N) in enumerate(mlp_shapes(DECODE_3B["hidden"], DECODE_3B["ffn"])):
            c = make_linear_case(M, K, N, DECODE_3B["r"], DECODE_3B["E"],
                                 seed=seed * 1024 + layer * 4 + i, exact_quota=False, with_grad=False)
            c["name"] = f"L{layer}.{name}"
            cases.append(c)
    return cases


def decode_activations(M: int, K: int, E: int, seed: int, plant: float = 6.0) -> dict:
    """Activations and router of one decode linear without the (large) weight draws:
    X [M,K] ~ N(0,1) bf16 with a Zipf(1.1) expert planted per token (i.i.d. draws), Wr [E,K] orthonormal rows."""
    rr = _rng(seed, 4)
    Wr = router_weights(E, K, rr, orthonormal=True)
    planted = zipf_assignment(M, E, rr, exact_quota=False)
    X = _rng(seed, 0).standard_normal((M, K), dtype=np.float32) + np.float32(plant) * Wr[planted]
    return dict(X=bf16_values(X), Wr=Wr, planted=planted)
