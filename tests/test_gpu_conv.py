"""Factorised 3 x 3 convolution on NHWC activations (im2col rows never formed, col2im folded into dX) against the
CPU checker applied to host-materialised rows, through the C-ABI."""
import numpy as np
import pytest
import torch

from oracle import ab_oracle as orc
from paper_2405_01067_b200 import synth

pytestmark = pytest.mark.gpu
TOL = 2e-2


@pytest.fixture(scope="module")
def ab():
    from paper_2405_01067_b200 import binding
    binding.lib()
    return binding


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda().to(torch.bfloat16)


def host(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def conv_case(seed, B, H, W, C, m, r):
    st = synth.streams(seed, ["AB", "x", "dY"])
    sigma = np.maximum(0.9 ** np.arange(r), 0.05) * (1.0 + 0.02 * (np.sqrt(m) + np.sqrt(9 * C)))
    A, Bf = synth.planted_factors(st["AB"], m, 9 * C, sigma, True)
    return dict(x=synth.half_normal(st["x"], (B, H, W, C), True), dY=synth.normal(st["dY"], (B, H, W, m), 1.0, True),
                A=A, B=Bf)


def check(ab, d, save_T=True):
    x, dY, A, Bf = (dev(d[k]) for k in ("x", "dY", "A", "B"))
    B, H, W, C = x.shape
    m, r = A.shape
    ws = ab.workspace(ab.ab_conv3x3_workspace_bytes(B, H, W, C, m, r), "cuda")
    y, T = ab.ab_conv3x3_forward(x, A, Bf, save_T=save_T, ws=ws)
    torch.cuda.synchronize()
    assert ab.workspace_status(ws) == 0
    dX, dA, dB = ab.ab_conv3x3_backward(x, dY, A, Bf, T_saved=T, ws=ws)
    dX2, dA2, dB2 = ab.ab_conv3x3_backward(x, dY, A, Bf, T_saved=T, ws=ws)
    torch.cuda.synchronize()
    assert ab.workspace_status(ws) == 0
    assert torch.equal(dA, dA2) and torch.equal(dB, dB2) and torch.equal(dX, dX2)
    T_ref, y_ref = orc.conv3x3_forward(d["x"], d["A"], d["B"])
    dX_ref, dA_ref, dB_ref, _ = orc.conv3x3_backward(d["x"], d["dY"].reshape(-1, m), d["A"], d["B"])
    pairs = dict(y=(host(y).reshape(-1, m), y_ref), dX=(host(dX).reshape(-1, C), dX_ref.reshape(-1, C)),
                 dA=(host(dA), dA_ref), dB=(host(dB), dB_ref))
    if T is not None:
        pairs["T"] = (host(T), T_ref)
    for k, (g, ref) in pairs.items():
        assert orc.rel_frob(g, ref) <= TOL, (k, orc.rel_frob(g, ref))
        assert orc.max_tile_rel_frob(g, ref) <= TOL, (k, "tile", orc.max_tile_rel_frob(g, ref))


@pytest.mark.parametrize("B,H,W,C,m,r", [
    (8, 4, 4, 64, 64, 16),        # eight whole images per tile (VGG-like 4 x 4)
    (3, 4, 4, 72, 40, 8),         # channels not a multiple of 64, ragged last group of images
    (5, 14, 14, 64, 128, 32),     # two tiles of 7 image rows per image (98 pixels: partial last group)
    (2, 14, 14, 256, 256, 128),   # the ResNet-50 layer3 shape, small batch
    (3, 7, 9, 24, 48, 24),        # odd image, one image per tile
    (2, 20, 12, 40, 64, 40),      # image taller than a tile: 2 tiles of 10 rows
    (20, 2, 2, 16, 16, 8),        # 32 tiny images per tile
    (1, 1, 1, 8, 8, 8),
    (4, 4, 4, 512, 512, 64),      # 512 input channels: two 256-channel windows of dX and of dB per tap
])
def test_conv3x3_shapes(ab, B, H, W, C, m, r):
    check(ab, conv_case(900 + B + H + C, B, H, W, C, m, r))


def test_conv3x3_recomputed_T_and_optional_outputs(ab):
    d = conv_case(950, 6, 8, 8, 64, 96, 24)
    x, dY, A, Bf = (dev(d[k]) for k in ("x", "dY", "A", "B"))
    y, T = ab.ab_conv3x3_forward(x, A, Bf, save_T=True)
    full = ab.ab_conv3x3_backward(x, dY, A, Bf, T_saved=T)
    rec = ab.ab_conv3x3_backward(x, dY, A, Bf, want=("dA",))
    only = ab.ab_conv3x3_backward(x, dY, A, Bf, want=("dX", "dB"))
    torch.cuda.synchronize()
    assert rec[0] is None and rec[2] is None and only[1] is None
    assert torch.equal(only[0], full[0]) and torch.equal(only[2], full[2])
    assert orc.rel_frob(host(rec[1]), host(full[1])) <= 1e-4


def test_conv3x3_unsupported_and_bad_arguments(ab):
    L = ab.lib()
    x = torch.zeros((2, 4, 4, 12), dtype=torch.bfloat16, device="cuda")      # C not a multiple of 8
    A = torch.zeros((16, 8), dtype=torch.bfloat16, device="cuda")
    Bf = torch.zeros((8, 108), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(ab.AbError) as e:
        ab.ab_conv3x3_forward(x, A, Bf)
    assert e.value.status in (ab.AB_ERR_UNSUPPORTED, ab.AB_ERR_INVALID_ARG)
    assert L.ab_conv3x3_workspace_bytes(0, 4, 4, 8, 8, 8) == 0


def test_conv3x3_full_size_resnet_and_vgg(ab):
    """ResNet-50 layer3 (batch 128, 14 x 14, 256 -> 256 channels, r = 128) and the VGG16 512-channel layer at 4 x 4
    (batch 1024, r = 32) at full size."""
    for (B, H, W, C, m, r) in [(128, 14, 14, 256, 256, 128), (1024, 4, 4, 512, 512, 32)]:
        check(ab, conv_case(970 + H, B, H, W, C, m, r))
