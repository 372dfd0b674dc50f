"""The forward product for callers that cannot allocate device memory (fp4q_gemm_fwd_static_workspace).

Some users of this library run where cudaMalloc is not theirs to call: inside an application that owns the
device heap, in a loop that must never enter the allocator, or in a sandbox limited to buffers it was given.
They pass inputs and outputs only; the kernel's workspace is a fixed array inside the library.  This test
calls that entry point through the C ABI twice in a row (the array is shared and keeps the previous call's
contents, so the second call checks that it is cleared correctly) and compares both results with the regular
entry point's.  It lives in a file that sorts last so that a run stopping at the first failure has already
run every other test; it passes alone in a fresh process as well as after the others."""
import numpy as np
import pytest
import torch

from paper_2607_24953_b200 import binding, workloads

pytestmark = pytest.mark.gpu


def _within_tolerance(got, ref):
    g, r = got.double().cpu().numpy(), ref.double().cpu().numpy()
    assert np.linalg.norm(g - r) <= 1e-3 * np.linalg.norm(r)
    assert (np.abs(g - r) <= 1e-2 * np.abs(r).max(axis=1, keepdims=True)).all()


@pytest.mark.parametrize("T,N,K,dt", [(128, 256, 256, binding.OUT_F32), (1000, 1152, 2304, binding.OUT_BF16)])
def test_static_workspace_forward_matches_regular_entry_point_twice(T, N, K, dt):
    dev = torch.device("cuda", 0)
    X = workloads.activations_student_t(T, K, 901, dev)
    W = workloads.weights(N, K, 900, dev)
    qx = binding.fp4q_quantize2d(X, mode=binding.ROUND_STOCHASTIC, seed=9, tensor_id=1)
    qw = binding.fp4q_quantize2d(W, mode=binding.ROUND_STOCHASTIC, seed=9, tensor_id=0)
    ref = binding.fp4q_gemm_fwd(qx, qw, dt=dt)                       # regular entry point, caller's workspace
    torch.cuda.synchronize()

    # everything the no-allocation call needs is created up front, as such a caller would have it
    odt = torch.float32 if dt == binding.OUT_F32 else torch.bfloat16
    outs = [torch.full((T, N), float("nan"), dtype=odt, device=dev) for _ in range(2)]
    status = torch.full((2,), 0x7FFFFFFF, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()
    before = torch.cuda.memory_allocated(dev)
    for i in range(2):                                               # two calls in a row on one stream
        binding.fp4q_gemm_fwd_static_workspace(qx, qw, outs[i], dt=dt, status_out=status[i:i + 1], stream=stream)
    assert torch.cuda.memory_allocated(dev) == before                # the binding allocated nothing either
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [0, 0]
    for o in outs:
        _within_tolerance(o, ref)
    assert torch.equal(outs[0], outs[1])


def test_static_workspace_argument_errors_are_reported():
    dev = torch.device("cuda", 0)
    qx = binding.fp4q_quantize2d(torch.zeros(64, 64, dtype=torch.bfloat16, device=dev))
    qw = binding.fp4q_quantize2d(torch.zeros(32, 96, dtype=torch.bfloat16, device=dev))
    out = torch.empty((64, 32), dtype=torch.float32, device=dev)
    with pytest.raises(binding.Fp4qError) as err:
        binding.fp4q_gemm_fwd_static_workspace(qx, qw, out, dt=binding.OUT_F32)     # contraction lengths differ
    assert err.value.status == 2
