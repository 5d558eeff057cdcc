"""Seeded synthetic inputs shaped like the layers AB-Training was evaluated on.

This module only draws random numbers and arranges them; it performs none of
the method's arithmetic (no factorisation, no averaging, no layer products), so
both the CUDA path and the CPU checker can take their inputs from it.

Every array is float32 (values of the bf16 workloads are rounded to bf16 here,
round-to-nearest-even, so that both sides see bit-identical numbers) and
C-contiguous.  Randomness: ``numpy.random.Generator(PCG64)`` with one child of
``SeedSequence(seed)`` per named tensor, spawned in a fixed order.

Workloads (Section "Experimental Evaluation" of the paper names the models;
only their layer shapes are used, the values are synthetic):

* ``linear_fp32``    one 256x512 linear layer, rank 32, 64 rows, K=2 groups
* ``vit_mlp``        ViT-B/16 MLP pair 3072x768 / 768x3072, rank 192, 50,432 rows, K=4
* ``resnet_conv``    ResNet-50 layer3 3x3 convolution as a GEMM, 256x2304, rank 128
* ``vit_sync``       the 72 weight matrices of ViT-B/16 with spectrum exp(-i/64), K=8
* ``vgg_conv``       VGG16 512x4608 convolution with planted rank 16, ranks 8..64
"""
from __future__ import annotations

import numpy as np

# std of N(0, 1e-3) and N(0, 1e-4): the second argument is read as a variance.
STD_GROUP_NOISE = float(np.sqrt(1e-3))
STD_VGG_NOISE = float(np.sqrt(1e-4))


def bf16_round(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result stays float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    u = (u + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of values that are already bf16-representable."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> np.uint32(16)).astype(np.uint16).reshape(a.shape)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    """float32 values of uint16 bf16 bit patterns (exact)."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).reshape(b.shape)


def streams(seed: int, names) -> dict:
    """One independent generator per name, children of SeedSequence(seed) in the given order."""
    kids = np.random.SeedSequence(seed).spawn(len(names))
    return {nm: np.random.Generator(np.random.PCG64(k)) for nm, k in zip(names, kids)}


def normal(rng, shape, std=1.0, bf16=False) -> np.ndarray:
    a = rng.standard_normal(shape, dtype=np.float32)
    if std != 1.0:
        a *= np.float32(std)
    return bf16_round(a) if bf16 else a


def half_normal(rng, shape, bf16=False) -> np.ndarray:
    """|N(0,1)|: stands in for post-ReLU activations."""
    a = np.abs(rng.standard_normal(shape, dtype=np.float32))
    return bf16_round(a) if bf16 else a


def orthonormal(rng, rows: int, cols: int) -> np.ndarray:
    """rows x cols matrix with orthonormal columns (QR of a Gaussian, float64, sign-fixed)."""
    g = rng.standard_normal((rows, cols))
    q, rr = np.linalg.qr(g)
    q *= np.sign(np.diag(rr))[None, :]
    return q


def planted_matrix(rng, m: int, n: int, sigma: np.ndarray) -> np.ndarray:
    """P diag(sigma) Q^T with random orthonormal P (m x s), Q (n x s); float32."""
    s = len(sigma)
    p = orthonormal(rng, m, s)
    q = orthonormal(rng, n, s)
    return np.ascontiguousarray((p * np.asarray(sigma, dtype=np.float64)[None, :]) @ q.T, dtype=np.float32)


def planted_factors(rng, m: int, n: int, sigma: np.ndarray, bf16=False):
    """A synthetic factor pair (A m x r, B r x n) with orthogonal columns/rows whose
    product has the planted singular values ``sigma``: the kind of input a trained
    factorised layer would hand to the kernels."""
    r = len(sigma)
    p = orthonormal(rng, m, r)
    q = orthonormal(rng, n, r)
    h = np.sqrt(np.asarray(sigma, dtype=np.float64))
    a = np.ascontiguousarray(p * h[None, :], dtype=np.float32)
    b = np.ascontiguousarray(h[:, None] * q.T, dtype=np.float32)
    if bf16:
        a, b = bf16_round(a), bf16_round(b)
    return a, b


def group_noise(seed: int, K: int, shape_a, shape_b, std=STD_GROUP_NOISE, bf16=False):
    """Per-group perturbations (E_k, E'_k), k = 0..K-1, independently seeded."""
    names = [f"noise_A{k}" for k in range(K)] + [f"noise_B{k}" for k in range(K)]
    st = streams(seed + 7919, names)
    ea = [normal(st[f"noise_A{k}"], shape_a, std, bf16) for k in range(K)]
    eb = [normal(st[f"noise_B{k}"], shape_b, std, bf16) for k in range(K)]
    return ea, eb


# --------------------------------------------------------------------------- workloads

def linear_fp32(seed: int = 0) -> dict:
    """256x512 layer, fp32, 64 rows, K=2.  Factors come from the caller's split of W at r=32."""
    m, n, r, N, K = 256, 512, 32, 64, 2
    st = streams(seed, ["W", "x", "dY"])
    ea, eb = group_noise(seed, K, (m, r), (r, n))
    return dict(name="linear_fp32", dtype="f32", m=m, n=n, r=r, N=N, K=K,
                W=normal(st["W"], (m, n), float(np.sqrt(1.0 / 512))),
                x=normal(st["x"], (N, n)), dY=normal(st["dY"], (N, m)),
                noise_A=ea, noise_B=eb)


def vit_mlp_weights(seed: int = 1, scale: int = 1) -> dict:
    """W1 3072x768 and W2 768x3072: 0.02*G plus a planted spectrum 0.9^i (fp32).
    ``scale`` divides both dimensions (tests use scaled-down copies of the recipe)."""
    big, small = 3072 // scale, 768 // scale
    st = streams(seed, ["W1g", "W1p", "W2g", "W2p"])
    sig = 0.9 ** np.arange(small)
    w1 = normal(st["W1g"], (big, small), 0.02) + planted_matrix(st["W1p"], big, small, sig)
    w2 = normal(st["W2g"], (small, big), 0.02) + planted_matrix(st["W2p"], small, big, sig)
    return dict(W1=w1, W2=w2)


def chain_case(seed: int, m: int, n: int, r: int, N: int, K: int = 1, bf16: bool = True,
               x_kind: str = "normal", sigma=None, want_dY: bool = True) -> dict:
    """Inputs of one factorised layer step: x (N x n), dY (N x m), a planted factor pair
    and K per-group perturbations of it."""
    st = streams(seed, ["AB", "x", "dY"])
    if sigma is None:
        # planted decay on top of a flat floor: a trained layer's leading spectrum
        sigma = np.maximum(0.9 ** np.arange(r), 0.05) * (1.0 + 0.02 * (np.sqrt(m) + np.sqrt(n)))
    a, b = planted_factors(st["AB"], m, n, sigma, bf16)
    x = half_normal(st["x"], (N, n), bf16) if x_kind == "half_normal" else normal(st["x"], (N, n), 1.0, bf16)
    out = dict(dtype="bf16" if bf16 else "f32", m=m, n=n, r=r, N=N, K=K, A=a, B=b, x=x)
    if want_dY:
        out["dY"] = normal(st["dY"], (N, m), 1.0, bf16)
    if K > 1:
        out["noise_A"], out["noise_B"] = group_noise(seed, K, (m, r), (r, n), STD_GROUP_NOISE, bf16)
    return out


def vit_mlp(layer: int = 1, seed: int = 1, N: int = 256 * 197, K: int = 4) -> dict:
    """ViT-B/16 MLP layer (1: 3072x768, 2: 768x3072), bf16, rank 192, batch 256 x 197 tokens."""
    m, n = (3072, 768) if layer == 1 else (768, 3072)
    d = chain_case(seed * 10 + layer, m, n, 192, N, K, True)
    d["name"] = f"vit_mlp_w{layer}"
    return d


def resnet_conv(seed: int = 2, N: int = 128 * 14 * 14) -> dict:
    """ResNet-50 layer3 3x3 convolution as im2col GEMM: W 256x2304 Kaiming-normal, r=128,
    rows are |N(0,1)| (materialised im2col rows), bf16."""
    m, n, r = 256, 2304, 128
    st = streams(seed, ["W"])
    d = chain_case(seed * 10, m, n, r, N, 1, True, x_kind="half_normal",
                   sigma=np.sqrt(2.0 / n) * (np.sqrt(n) + np.sqrt(m) * np.linspace(1.0, 0.0, r)))
    d["W"] = normal(st["W"], (m, n), float(np.sqrt(2.0 / n)))
    d["name"] = "resnet_conv"
    return d


VIT_BLOCK_SHAPES = [(768, 768)] * 4 + [(3072, 768), (768, 3072)]


def vit_sync_shapes(blocks: int = 12):
    return [s for _ in range(blocks) for s in VIT_BLOCK_SHAPES]


def vit_sync_matrix(seed: int, index: int, m: int, n: int, K: int = 8, scale: int = 1) -> dict:
    """One matrix of the ViT-B/16 group sync: planted factors with sigma_i = exp(-i/64),
    i < r = min(m,n)/4, and K noisy copies' perturbations.  ``scale`` divides the shape
    (tests use scaled-down copies of the same recipe)."""
    m, n = m // scale, n // scale
    r = min(m, n) // 4
    st = streams(seed * 1000 + index, ["AB"])
    sig = np.exp(-np.arange(r) / 64.0)
    a, b = planted_factors(st["AB"], m, n, sig)
    ea, eb = group_noise(seed * 1000 + index, K, (m, r), (r, n))
    return dict(name=f"vit_sync_{index}", dtype="f32", m=m, n=n, r=r, K=K, A=a, B=b,
                noise_A=ea, noise_B=eb, sigma=sig)


def vgg_conv(r: int, seed: int = 4, N: int = 1024 * 16, K: int = 4) -> dict:
    """VGG16 512x4608 convolution as GEMM, bf16.  W = (0.02/4) G1(512x16) G2(16x4608) + N(0,1e-4)."""
    m, n = 512, 4608
    st = streams(seed, ["G1", "G2", "Wn"])
    g1 = st["G1"].standard_normal((m, 16))
    g2 = st["G2"].standard_normal((16, n))
    w = np.ascontiguousarray((0.02 / 4) * (g1 @ g2), dtype=np.float32) + normal(st["Wn"], (m, n), STD_VGG_NOISE)
    sig = np.concatenate([np.linspace(8.0, 6.0, 16), np.full(48, 0.85)])[:r]
    d = chain_case(seed * 10 + r, m, n, r, N, K, True, sigma=sig)
    d["W"] = w
    d["name"] = f"vgg_conv_r{r}"
    return d


def group_copies(base: np.ndarray, noise, bf16: bool = False) -> np.ndarray:
    """Stack the K perturbed copies base + noise[k] into one (K, ...) array (input assembly only)."""
    out = np.stack([base + e for e in noise]).astype(np.float32)
    return bf16_round(out) if bf16 else np.ascontiguousarray(out)
