"""sysconv1d_host_static: the host-buffer convolution for callers that may not allocate device memory.

Some users of this library run where cudaMalloc is off limits (a plug-in inside an application that
owns all device memory, a real-time loop with an allocation ban), so they cannot hand sysconv1d_host
the device workspace it needs.  The static variant stages through a fixed array inside the library.
This test calls it through the C ABI twice in a row -- the second call on a shorter, different signal
with another design, so stale contents of the shared array would show -- and compares each result with
what sysconv1d_host returns for the same inputs (same kernel, so the two must agree bit for bit) and
with the CPU oracle (within the tolerance of the parity tests).

Collected last on purpose: a failure here must not hide the other tests behind `-x`.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2010_15884_b200 import binding as B
from paper_2010_15884_b200 import inputs

pytestmark = pytest.mark.gpu

TOL = 1e-5


def _both_ways(x, w, design, device):
    n, q = x.shape[-1], w.shape[0]
    xh = torch.from_numpy(x).pin_memory()
    shape = x.shape[:-1] + (n - q + 1,)
    y_static = torch.full(shape, float("nan"), dtype=torch.float32).pin_memory()
    y_plain = torch.full(shape, float("nan"), dtype=torch.float32).pin_memory()
    B.sysconv1d_host_static(xh, w, y_static, design)
    torch.cuda.synchronize()
    work = torch.empty(B.host_workspace_bytes(tuple(x.shape), (q,)), dtype=torch.uint8, device=device)
    B.sysconv1d_host(xh, w, y_plain, design, work)
    torch.cuda.synchronize()
    a, b = y_static.numpy().astype(np.float64), y_plain.numpy().astype(np.float64)
    assert np.isfinite(a).all() and np.isfinite(b).all()
    # against the existing entry point: within the tolerance of the parity tests, 1e-5 * sum |w||x| per output
    # (both run the same kernel on the same data, so in fact every bit must agree)
    ref = [oracle.conv1d_f32(row, w) for row in x.reshape(-1, n)]
    y_ref = np.stack([r[0] for r in ref]).reshape(shape)
    scale = np.stack([r[1] for r in ref]).reshape(shape)
    assert np.all(np.abs(a - b) <= TOL * scale)
    assert np.array_equal(y_static.numpy(), y_plain.numpy())
    # against the definition (Eq. 2), computed by the CPU oracle
    assert np.all(np.abs(a - y_ref) <= TOL * scale)


def test_static_variant_matches_workspace_variant_twice_in_a_row(cuda_device):
    x1, ws1 = inputs.gen_1d_f32(300000, [16], seed=71)
    _both_ways(x1, ws1[16], B.OS, cuda_device)
    # second call: shorter batched signals, other data, other design -- the array still holds call 1
    rng = np.random.default_rng(72)
    x2 = (rng.random((3, 40001), dtype=np.float32) * 2 - 1).astype(np.float32)
    w2 = (rng.random(5, dtype=np.float32) * 2 - 1).astype(np.float32)
    _both_ways(x2, w2, B.IS, cuda_device)


def test_static_variant_rejects_what_does_not_fit(cuda_device):
    cap = B.static_scratch_bytes()
    assert cap == 16 << 20
    n = cap // 8 + 1024                      # x and y together exceed the area
    xh = torch.zeros(n, dtype=torch.float32).pin_memory()
    yh = torch.zeros(n - 3, dtype=torch.float32).pin_memory()
    before = B.launch_count()
    with pytest.raises(B.SysconvError) as e:
        B.sysconv1d_host_static(xh, np.ones(4, np.float32), yh, B.OS)
    assert e.value.status == 5
    assert B.launch_count() == before        # nothing was enqueued
