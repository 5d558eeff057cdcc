"""CPU checker for the AB-Training hot path.  TEST INFRASTRUCTURE, NOT THE PRODUCT.

Plain float64 numpy, written from the paper's definitions; it shares no code
with the CUDA path and must never be imported by the package.  Only the test
suite, the smoke check and the benchmark's CPU-baseline leg call it.

What each function follows:

* ``forward`` / ``backward``   the layer W = A B of Eq. 3 used as a linear map
  y = x W^T, and the chain rule through the rank-r intermediate.
* ``im2col_3x3`` / ``col2im_3x3`` / ``conv3x3_*``  the flattening of a convolution weight's
  trailing dimensions (Methodology, after Eq. 3) applied to NHWC activations.
* ``dense_forward`` / ``dense_backward``  the same layer with W dense (Algorithm 1's
  full-rank steps: warm-up and rebound).
* ``group_average*``           Algorithm 1, the two allReduce(./worldSize) lines.
* ``recombine``                Algorithm 1, "W <- AB".
* ``jacobi_svd``               the SVD that Eq. 3 refers to (one-sided Jacobi,
  run to 1e-14 relative off-orthogonality).
* ``rank_rule``                Section "Methodology", AB-decomposition bullet:
  singular values below sigmaCutoff times the largest are dropped.
* ``svd_split``                Eq. 3: A = U S^(1/2), B = S^(1/2) V^T.

Pins (tests/test_oracle_*.py): finite differences, the dense restatement,
Eckart-Young, exact recovery at rank <= r, closed-form singular values,
LAPACK, planted spectra, bit-level properties of the fixed-order fp32 mean,
hand-computed values of the two error yardsticks (``rel_frob``,
``max_tile_rel_frob``).  No function here is "parity unpinned".
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


def _f64(a):
    return np.asarray(a, dtype=F64)


# ------------------------------------------------------------------ layer (Eq. 3)

def forward(x, A, B):
    """T = x B^T (N x r), y = T A^T (N x m).  Eq. 3 with W = A B applied as y = x W^T."""
    x, A, B = _f64(x), _f64(A), _f64(B)
    T = x @ B.T
    y = T @ A.T
    return T, y


def backward(x, dY, A, B):
    """Chain rule of L(y) through y = (x B^T) A^T given dY = dL/dy.

    dT = dY A, dX = dT B, dA = dY^T T, dB = dT^T x.  Returns (dX, dA, dB, dT)."""
    x, dY, A, B = _f64(x), _f64(dY), _f64(A), _f64(B)
    T = x @ B.T
    dT = dY @ A
    dX = dT @ B
    dA = dY.T @ T
    dB = dT.T @ x
    return dX, dA, dB, dT


def im2col_3x3(x):
    """Rows of a 3 x 3 convolution with stride 1 and zero padding 1 over an NHWC activation x [B, H, W, C]:
    row (b, oy, ox) holds x[b, oy + ky - 1, ox + kx - 1, c] at column (ky * 3 + kx) * C + c (zeros outside
    the image).  This is the flattening of the trailing weight dimensions (Methodology, after Eq. 3) seen
    from the activation side: a convolution weight [m, ky, kx, C] flattened to m x 9C multiplies these rows."""
    x = _f64(x)
    B, H, W, C = x.shape
    xp = np.zeros((B, H + 2, W + 2, C))
    xp[:, 1:H + 1, 1:W + 1] = x
    rows = np.empty((B, H, W, 9, C))
    for ky in range(3):
        for kx in range(3):
            rows[:, :, :, ky * 3 + kx] = xp[:, ky:ky + H, kx:kx + W]
    return rows.reshape(B * H * W, 9 * C)


def col2im_3x3(rows, B, H, W, C):
    """The transpose of ``im2col_3x3``: every entry of a row is added back to the pixel it was taken from
    (entries taken from the padding are dropped).  Turns the gradient of the rows into that of x."""
    r = _f64(rows).reshape(B, H, W, 9, C)
    xp = np.zeros((B, H + 2, W + 2, C))
    for ky in range(3):
        for kx in range(3):
            xp[:, ky:ky + H, kx:kx + W] += r[:, :, :, ky * 3 + kx]
    return xp[:, 1:H + 1, 1:W + 1].copy()


def conv3x3_forward(x, A, B):
    """Factorised 3 x 3 convolution: the layer of Eq. 3 applied to the im2col rows.  Returns (T, y) as
    [pixels, r] and [pixels, m]."""
    return forward(im2col_3x3(x), A, B)


def conv3x3_backward(x, dY, A, B):
    """Chain rule of the factorised convolution.  Returns (dX [B,H,W,C], dA, dB, dT)."""
    Bn, H, W, C = np.shape(x)
    dXr, dA, dB, dT = backward(im2col_3x3(x), dY, A, B)
    return col2im_3x3(dXr, Bn, H, W, C), dA, dB, dT


def dense_forward(x, W):
    """y = x W^T: the layer with W held dense (Algorithm 1's full-rank steps before the first decomposition
    and after W <- A B)."""
    return _f64(x) @ _f64(W).T


def dense_backward(x, dY, W):
    """Chain rule of L(y) through y = x W^T: dX = dY W, dW = dY^T x.  Returns (dX, dW)."""
    x, dY, W = _f64(x), _f64(dY), _f64(W)
    return dY @ W, dY.T @ x


# ------------------------------------------------------------------ group mean (Algorithm 1)

def group_average(copies):
    """Exact (float64) mean over the leading axis of K stacked copies."""
    c = _f64(copies)
    return c.sum(axis=0) / c.shape[0]


def group_average_f32(copies):
    """The mean as fp32 arithmetic in a fixed order: s = c0; s = fl(s + c_k) for k = 1..K-1;
    out = fl(s * fl(1/K)).  Inputs are float32 values (bf16 inputs widen exactly)."""
    c = np.asarray(copies, dtype=np.float32)
    K = c.shape[0]
    s = c[0].copy()
    for k in range(1, K):
        s = (s + c[k]).astype(np.float32)
    inv = np.float32(1.0) / np.float32(K)
    return (s * inv).astype(np.float32)


def group_average_prescaled_f32(copies):
    """Algorithm 1 as printed: each copy is divided by the number of workers, then summed."""
    c = np.asarray(copies, dtype=np.float32)
    K = c.shape[0]
    s = (c[0] / np.float32(K)).astype(np.float32)
    for k in range(1, K):
        s = (s + (c[k] / np.float32(K)).astype(np.float32)).astype(np.float32)
    return s


def recombine(Abar, Bbar):
    """W = A B (Algorithm 1, the loop after the two all-reduces)."""
    return _f64(Abar) @ _f64(Bbar)


# ------------------------------------------------------------------ SVD (Eq. 3)

def _round_robin(n):
    """The rounds of disjoint index pairs that together cover every pair (i < j < n) once."""
    idx = list(range(n + (n & 1)))
    rounds = []
    for _ in range(len(idx) - 1):
        half = len(idx) // 2
        p = np.array(idx[:half])
        q = np.array(idx[half:][::-1])
        keep = (p < n) & (q < n)
        rounds.append((np.minimum(p, q)[keep], np.maximum(p, q)[keep]))
        idx = [idx[0]] + [idx[-1]] + idx[1:-1]
    return rounds


def jacobi_svd(W, tol=1e-14, max_sweeps=60):
    """Thin SVD W = U diag(s) V^T by one-sided (Hestenes) Jacobi in float64.

    Columns of the shorter side are orthogonalised by plane rotations until every
    pair satisfies |a_i.a_j| <= tol |a_i||a_j|; the paper's remark that W is
    transposed when n > m is this choice of side and does not change the result.
    Columns whose norm falls below eps * largest are treated as zero.
    Returns U (m x s), s descending (s,), Vt (s x n), sweeps."""
    W = _f64(W)
    m, n = W.shape
    if n > m:
        U, s, Vt, sw = jacobi_svd(W.T, tol, max_sweeps)
        return Vt.T.copy(), s, U.T.copy(), sw
    G = W.copy()                       # m x n, columns get orthogonalised
    V = np.eye(n)
    rounds = _round_robin(n)
    tiny = np.finfo(F64).eps
    sweeps = 0
    for sweeps in range(1, max_sweeps + 1):
        worst = 0.0
        big = float(np.einsum("ij,ij->j", G, G).max(initial=0.0))   # largest squared column norm
        for p, q in rounds:
            if p.size == 0:
                continue
            gp, gq = G[:, p], G[:, q]
            alpha = np.einsum("ij,ij->j", gp, gp)
            beta = np.einsum("ij,ij->j", gq, gq)
            gamma = np.einsum("ij,ij->j", gp, gq)
            live = (alpha > (tiny * tiny) * big) & (beta > (tiny * tiny) * big) & (gamma != 0.0)
            denom = np.sqrt(np.where(live, alpha * beta, 1.0))
            off = np.where(live, np.abs(gamma) / denom, 0.0)
            worst = max(worst, float(off.max(initial=0.0)))
            rot = live & (off > tol)
            if not rot.any():
                continue
            g = np.where(rot, gamma, 1.0)
            zeta = (beta - alpha) / (2.0 * g)
            t = np.sign(zeta) / (np.abs(zeta) + np.sqrt(1.0 + zeta * zeta))
            t = np.where(zeta == 0.0, 1.0, t)
            c = 1.0 / np.sqrt(1.0 + t * t)
            s_ = c * t
            c = np.where(rot, c, 1.0)
            s_ = np.where(rot, s_, 0.0)
            G[:, p], G[:, q] = c * gp - s_ * gq, s_ * gp + c * gq
            vp, vq = V[:, p], V[:, q]
            V[:, p], V[:, q] = c * vp - s_ * vq, s_ * vp + c * vq
        if worst <= tol:
            break
    s = np.sqrt(np.einsum("ij,ij->j", G, G))
    order = np.argsort(-s, kind="stable")
    s = s[order]
    G = G[:, order]
    V = V[:, order]
    U = np.zeros_like(G)
    nz = s > tiny * (s[0] if s.size and s[0] > 0 else 1.0)
    U[:, nz] = G[:, nz] / s[nz]
    return U, s, V.T.copy(), sweeps


def rank_rule(sigma, sigma_cutoff, r_max):
    """Kept rank: the count of sigma_i >= sigma_cutoff * sigma_1 (values smaller than the
    largest times the cutoff are removed), at most r_max and at least 1."""
    sigma = _f64(sigma)
    if sigma.size == 0:
        return 0
    keep = int(np.count_nonzero(sigma >= sigma_cutoff * sigma[0]))
    return max(1, min(int(r_max), keep))


def svd_split(W, r_max, sigma_cutoff=0.0):
    """Eq. 3 with the rank rule: A = U_r diag(sqrt s_r), B = diag(sqrt s_r) V_r^T.

    Returns A (m x r'), B (r' x n), all singular values (descending), r'."""
    U, s, Vt, _ = jacobi_svd(W)
    r = rank_rule(s, sigma_cutoff, min(int(r_max), s.size))
    h = np.sqrt(s[:r])
    A = U[:, :r] * h[None, :]
    B = h[:, None] * Vt[:r]
    return A, B, s, r


# ------------------------------------------------------------------ whole step

def group_sync(A_copies, B_copies, r_max, sigma_cutoff):
    """Algorithm 1 from the all-reduces to the next decomposition: mean of the K copies of A
    and B, W = Abar Bbar, split of W under the rank rule.  Returns dict of all pieces."""
    Abar = group_average(A_copies)
    Bbar = group_average(B_copies)
    W = recombine(Abar, Bbar)
    A, B, s, r = svd_split(W, r_max, sigma_cutoff)
    return dict(Abar=Abar, Bbar=Bbar, W=W, A=A, B=B, sigma=s, r=r)


def adamw_step(p, g, m, v, lr, step, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=1e-2):
    """One AdamW update with decoupled weight decay (the optimizer of the paper's experiments), float64:
    p <- p (1 - lr wd); m <- b1 m + (1 - b1) g; v <- b2 v + (1 - b2) g^2;
    p <- p - lr (m / (1 - b1^t)) / (sqrt(v / (1 - b2^t)) + eps).  Returns new (p, m, v)."""
    p, g, m, v = _f64(p), _f64(g), _f64(m), _f64(v)
    p = p * (1.0 - lr * weight_decay)
    m = beta1 * m + (1.0 - beta1) * g
    v = beta2 * v + (1.0 - beta2) * g * g
    mhat = m / (1.0 - beta1 ** step)
    vhat = v / (1.0 - beta2 ** step)
    return p - lr * mhat / (np.sqrt(vhat) + eps), m, v


def lr_rebound_factor(steps_since_change, rebound_steps, floor=0.0):
    """Learning-rate rebound (Methodology): the rate restarts at `floor` of its scheduled value when the
    parameters change shape and climbs back linearly over rebound_steps steps (the paper gives no shape)."""
    if rebound_steps <= 0 or steps_since_change >= rebound_steps:
        return 1.0
    return floor + (1.0 - floor) * max(0, steps_since_change) / rebound_steps


def rel_frob(a, b):
    """||a - b||_F / ||b||_F in float64 (0 when both are zero)."""
    a, b = _f64(a), _f64(b)
    den = np.linalg.norm(b)
    num = np.linalg.norm(a - b)
    return 0.0 if num == 0.0 else num / den


def max_tile_rel_frob(a, b, tile_rows=128, tile_cols=64):
    """Largest relative Frobenius error over the tiles of a grid laid on the matrices:
    max over tiles of ||a_tile - b_tile||_F / max(||b_tile||_F, floor), where the floor is the norm a tile
    of that size would have at 1e-3 of b's root-mean-square value (so that a tile of b that happens to be
    all zeros does not divide by zero).  A wrong tile cannot hide behind the norm of the whole matrix."""
    a, b = _f64(a), _f64(b)
    if b.size == 0:
        return 0.0
    rms = np.sqrt(np.mean(b * b))
    ri = np.arange(0, b.shape[0], tile_rows)
    ci = np.arange(0, b.shape[1], tile_cols)

    def tile_sums(sq):          # sum of the entries of every tile
        return np.add.reduceat(np.add.reduceat(sq, ri, axis=0), ci, axis=1)

    num = np.sqrt(tile_sums((a - b) ** 2))
    den = np.sqrt(tile_sums(b * b))
    sizes = np.outer(np.diff(np.append(ri, b.shape[0])), np.diff(np.append(ci, b.shape[1])))
    den = np.maximum(den, 1e-3 * rms * np.sqrt(sizes))
    with np.errstate(divide="ignore", invalid="ignore"):
        rel = np.where(num > 0.0, num / den, 0.0)
    worst = rel.max()
    return float(worst)

