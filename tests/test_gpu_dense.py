"""Dense layer of the full-rank phases (y = x W^T, dX = dY W, dW = dY^T x) against the CPU checker, through
the C-ABI: bf16 storage on the tensor cores, fp32 storage and odd shapes on the general kernel."""
import numpy as np
import pytest
import torch

from oracle import ab_oracle as orc
from paper_2405_01067_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ab():
    from paper_2405_01067_b200 import binding
    binding.lib()
    return binding


def dev(a, bf16):
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()
    return t.to(torch.bfloat16) if bf16 else t


def host(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def dense_case(seed, N, m, n, bf16):
    st = synth.streams(seed, ["x", "dY", "W"])
    return dict(x=synth.normal(st["x"], (N, n), 1.0, bf16), dY=synth.normal(st["dY"], (N, m), 1.0, bf16),
                W=synth.normal(st["W"], (m, n), float(1.0 / np.sqrt(n)), bf16))


def check(ab, d, bf16):
    tol = 2e-2 if bf16 else 1e-4
    x, dY, W = (dev(d[k], bf16) for k in ("x", "dY", "W"))
    N, n = x.shape
    m = W.shape[0]
    code = ab.AB_BF16 if bf16 else ab.AB_F32
    ws_f = ab.workspace(ab.ab_workspace_bytes(ab.AB_OP_DENSE_FORWARD, N, m, n, 0, 1, code), "cuda")
    ws_b = ab.workspace(ab.ab_workspace_bytes(ab.AB_OP_DENSE_BACKWARD, N, m, n, 0, 1, code), "cuda")
    y = ab.ab_dense_forward(x, W, ws=ws_f)
    dX, dW = ab.ab_dense_backward(x, dY, W, ws=ws_b)
    dX2, dW2 = ab.ab_dense_backward(x, dY, W, ws=ws_b)
    torch.cuda.synchronize()
    assert ab.workspace_status(ws_f) == 0 and ab.workspace_status(ws_b) == 0
    assert torch.equal(dW, dW2) and torch.equal(dX, dX2)          # fixed order of the sums over the rows
    y_ref = orc.dense_forward(d["x"], d["W"])
    dX_ref, dW_ref = orc.dense_backward(d["x"], d["dY"], d["W"])
    for name, got, ref in (("y", y, y_ref), ("dX", dX, dX_ref), ("dW", dW, dW_ref)):
        g = host(got)
        assert orc.rel_frob(g, ref) <= tol, (name, orc.rel_frob(g, ref))
        assert orc.max_tile_rel_frob(g, ref) <= tol, (name, "tile", orc.max_tile_rel_frob(g, ref))
    only_x = ab.ab_dense_backward(x, dY, W, want=("dX",), ws=ws_b)
    only_w = ab.ab_dense_backward(x, dY, W, want=("dW",), ws=ws_b)
    torch.cuda.synchronize()
    assert only_x[1] is None and only_w[0] is None
    assert torch.equal(only_x[0], dX) and torch.equal(only_w[1], dW)


@pytest.mark.parametrize("N,m,n", [(300, 256, 128), (1000, 768, 256), (129, 136, 264), (77, 40, 56), (5000, 512, 1024),
                                   (64, 8, 8), (4100, 264, 776)])
def test_dense_bf16(ab, N, m, n):
    check(ab, dense_case(500 + N, N, m, n, True), True)


@pytest.mark.parametrize("N,m,n", [(64, 256, 512), (37, 19, 23), (130, 70, 66), (1, 1, 1)])
def test_dense_fp32(ab, N, m, n):
    check(ab, dense_case(600 + N, N, m, n, False), False)


def test_dense_bf16_odd_shape_takes_general_kernel(ab):
    check(ab, dense_case(700, 100, 50, 70, True), True)


def test_dense_empty_batch(ab):
    W = torch.randn(8, 6, device="cuda")
    x = torch.empty((0, 6), device="cuda")
    dY = torch.empty((0, 8), device="cuda")
    y = ab.ab_dense_forward(x, W)
    dX, dW = ab.ab_dense_backward(x, dY, W)
    torch.cuda.synchronize()
    assert y.shape == (0, 8) and dX.shape == (0, 6) and torch.count_nonzero(dW) == 0


def test_dense_vit_mlp_full_size(ab):
    """The dense W1 layer (3072 x 768) at 50,432 rows: y, dX over all rows in chunks, dW over all rows."""
    N, m, n = 256 * 197, 3072, 768
    d = dense_case(800, N, m, n, True)
    x, dY, W = (dev(d[k], True) for k in ("x", "dY", "W"))
    y = ab.ab_dense_forward(x, W)
    dX, dW = ab.ab_dense_backward(x, dY, W)
    torch.cuda.synchronize()
    dW_ref = np.zeros((m, n))
    for s in range(0, N, 8192):
        e = min(N, s + 8192)
        y_ref = orc.dense_forward(d["x"][s:e], d["W"])
        dX_ref, dWc = orc.dense_backward(d["x"][s:e], d["dY"][s:e], d["W"])
        dW_ref += dWc
        for name, got, ref in (("y", y, y_ref), ("dX", dX, dX_ref)):
            g = host(got[s:e])
            assert orc.rel_frob(g, ref) <= 2e-2 and orc.max_tile_rel_frob(g, ref) <= 2e-2, (name, s)
    assert orc.rel_frob(host(dW), dW_ref) <= 2e-2 and orc.max_tile_rel_frob(host(dW), dW_ref) <= 2e-2
