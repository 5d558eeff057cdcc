"""ab_layer_forward_static: the forward call for users who cannot allocate device memory (a
plug-in inside an application that owns the whole memory pool, a loop that must not touch
cudaMalloc).  Its scratch is an array built into the library, so the test checks what such a
user relies on: the result equals ab_layer_forward's and the CPU checker's, a second call right
after the first is not disturbed by what the first left in the shared array, the device's free
memory does not move across the calls, and a size beyond the built-in array is refused instead
of overrunning it.
Collected last on purpose: a failure here cannot hide another test's result."""
import ctypes

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


def _dev(a, bf16):
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()
    return t.to(torch.bfloat16) if bf16 else t


def _rel(a, b):
    a, b = a.double(), b.double()
    return float((a - b).norm() / b.norm())


@pytest.mark.parametrize("bf16,tol", [(False, 1e-4), (True, 2e-2)])
def test_two_calls_in_a_row_match_the_workspace_entry_point(ab, bf16, tol):
    cases = [synth.chain_case(31, 200, 176, 48, 900, bf16=bf16, want_dY=False),     # fills 43,200 scratch entries
             synth.chain_case(32, 96, 120, 16, 333, bf16=bf16, want_dY=False)]      # smaller: stale entries remain
    outs, refs = [], []
    tensors = [[_dev(d[k], bf16) for k in ("x", "A", "B")] for d in cases]
    ys = [torch.empty((d["N"], d["m"]), dtype=t[0].dtype, device="cuda") for d, t in zip(cases, tensors)]
    # one call first: loading the kernels and the first look-up of the array's address are behind us
    ab.ab_layer_forward_static(*tensors[1], ys[1])
    torch.cuda.synchronize()
    ys[1].zero_()
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]      # the driver's own count of free bytes on the device
    torch_before = torch.cuda.memory_allocated()
    for (x, A, B), y in zip(tensors, ys):          # back to back on one stream, no sync in between
        outs.append(ab.ab_layer_forward_static(x, A, B, y))
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before     # no cudaMalloc / cudaFree behind the calls
    assert torch.cuda.memory_allocated() == torch_before   # and nothing through torch's allocator
    for (x, A, B) in tensors:
        refs.append(ab.ab_layer_forward(x, A, B)[0])
    torch.cuda.synchronize()
    for got, ref, d in zip(outs, refs, cases):
        assert _rel(got, ref) <= tol
        y_ref = orc.forward(d["x"], d["A"], d["B"])[1]
        g = got.float().cpu().numpy()
        assert orc.rel_frob(g, y_ref) <= tol and orc.max_tile_rel_frob(g, y_ref) <= tol


def test_size_limit_and_bad_arguments(ab):
    L = ab.lib()
    cap = int(L.ab_static_scratch_elems())
    assert cap == 1 << 20
    p = ctypes.c_void_p(256)      # never dereferenced: the calls below are rejected on the host
    N = cap // 64 + 1             # N * r just beyond the array
    assert L.ab_layer_forward_static(p, p, p, p, N, 128, 128, 64, 64, 128, 0, None) == ab.AB_ERR_UNSUPPORTED
    # a row count whose product with r does not fit 64 bits must not slip under the limit
    assert L.ab_layer_forward_static(p, p, p, p, (2 ** 63 - 1) // 2, 128, 128, 64, 64, 128, 0, None) == ab.AB_ERR_UNSUPPORTED
    assert L.ab_layer_forward_static(p, p, p, p, 2 ** 58, 128, 128, 64, 64, 128, 0, None) == ab.AB_ERR_UNSUPPORTED
    assert L.ab_layer_forward_static(None, p, p, p, 8, 128, 128, 64, 64, 128, 0, None) == ab.AB_ERR_INVALID_ARG
    assert L.ab_layer_forward_static(p, p, p, p, 8, 128, 128, 200, 200, 128, 0, None) == ab.AB_ERR_INVALID_ARG
    # exactly at the limit is accepted and correct
    d = synth.chain_case(33, 64, 80, 64, cap // 64, bf16=True, want_dY=False)
    x, A, B = (_dev(d[k], True) for k in ("x", "A", "B"))
    y = torch.empty((d["N"], 64), dtype=torch.bfloat16, device="cuda")
    ab.ab_layer_forward_static(x, A, B, y)
    ref = ab.ab_layer_forward(x, A, B)[0]
    torch.cuda.synchronize()
    assert _rel(y, ref) <= 2e-2
    assert orc.rel_frob(y.float().cpu().numpy(), orc.forward(d["x"], d["A"], d["B"])[1]) <= 2e-2
