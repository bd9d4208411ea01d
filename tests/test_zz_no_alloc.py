"""The entry point for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is not an option: on a device whose memory was handed
out once at start-up, inside an application that keeps all device memory in its own pool, or in a loop
that cannot afford the device-wide synchronisation an allocation implies.  bsr_linear_backward_static
serves them by keeping its split-reduction scratch in a fixed array inside the library.  This test calls
it through the C ABI twice in a row (the second call finds the first call's leftovers in the shared
scratch) and checks both results against bsr_linear_backward, which takes its scratch from the caller,
and against the oracle's definition of the two gradients (Eq. 2 and Eq. 4).
It is collected last so that a run stopping at the first failure has already run everything else.
"""
import numpy as np
import pytest

from oracle import bsr_oracle as O
from paper_2405_10951_b200 import synth

pytestmark = pytest.mark.gpu


def rel(a, b):
    return float((a.double() - b.double()).norm() / b.double().norm())


def test_static_scratch_backward_matches_caller_scratch_backward_twice():
    import torch
    from paper_2405_10951_b200 import binding as Bd
    rng = np.random.default_rng(7)
    g = lambda a: torch.as_tensor(a.astype(np.float32)).cuda().to(torch.bfloat16)
    ws = torch.empty(160 * 128 * 256, dtype=torch.float32, device="cuda")
    # The first call on a device does the one-off set-up; with CUDA's lazy module loading that is also when the
    # device image holding the 16 MiB array is loaded, so the driver's free-memory figure drops by that much once.
    z = torch.zeros((8, 8), dtype=torch.bfloat16, device="cuda")
    Bd.bsr_linear_backward_static(z, z, z)
    torch.cuda.synchronize()
    # two different shapes back to back: the second call reuses the scratch the first one filled
    for m, n, k in [(9216, 768, 768), (3072, 384, 1536)]:
        xh, wh, dyh = (synth.round_to_bf16(a) for a in (rng.standard_normal((m, k)), rng.standard_normal((n, k)) / np.sqrt(k),
                                                        rng.standard_normal((m, n))))
        x, w, dy = g(xh), g(wh), g(dyh)
        dx_ref, dw_ref = Bd.bsr_linear_backward(x, w, dy, use_tensor_cores=True, workspace=ws)
        dx = torch.empty_like(dx_ref)
        dw = torch.empty_like(dw_ref)
        torch.cuda.synchronize()
        held = torch.cuda.memory_allocated()
        free_before = torch.cuda.mem_get_info()[0]            # the driver's view: a cudaMalloc by anyone would lower it
        Bd.bsr_linear_backward_static(x, w, dy, dx, dw)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == held          # the call itself took nothing from torch's pool ...
        assert torch.cuda.mem_get_info()[0] >= free_before    # ... and nothing from the device
        assert rel(dx, dx_ref) < 4e-3                         # tolerances of the other linear-backward tests
        assert rel(dw, dw_ref) < 1e-4
        dx_o, dw_o, _ = O.linear_bwd(dyh, xh, wh)             # and the definition itself
        assert rel(dx.cpu(), torch.as_tensor(dx_o)) < 4e-3
        assert rel(dw.cpu(), torch.as_tensor(dw_o)) < 1e-4


def test_static_scratch_rejects_oversized_weights():
    import torch
    from paper_2405_10951_b200 import binding as Bd
    m, n, k = 64, 2048, 2048          # n * k = 4 Mi elements: twice the documented limit
    x = torch.zeros((m, k), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((n, k), dtype=torch.bfloat16, device="cuda")
    dy = torch.zeros((m, n), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(Bd.BsrError) as e:
        Bd.bsr_linear_backward_static(x, w, dy)
    assert e.value.status == -3 and "exceeds the built-in scratch" in str(e.value)
