"""The GEMM kernels' bounded waits, exercised without faulting or hanging anything.

Every wait inside the kernels gives up after a number of polls, records FP4Q_ERR_TIMEOUT in the workspace and lets
the kernel leave through its normal exit.  Here that path is made to run: a development hook makes the first CTA
leave out one operand load (so the data a wait is waiting for never arrives) and the poll limit is set to a few
thousand, so the launch ends within milliseconds.  The test checks that the status is reported, that the process and
the CUDA context carry on, and that the next ordinary call on the same workspace is correct again."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_24953_b200 import binding, workloads
from tests.gpu_util import check_gemm, dequant_from_gpu

pytestmark = pytest.mark.gpu

FP4Q_ERR_TIMEOUT = 7


def _operands(T, N, K):
    X = workloads.activations_gauss_outliers(T, K, 101, "cuda")
    W = workloads.weights(N, K, 100, "cuda")
    return binding.fp4q_quantize2d(X), binding.fp4q_quantize2d(W)


@pytest.mark.parametrize("T,N,K,nth", [(128, 256, 256, 1),      # one CTA, one tile, one stage: its only load is withheld
                                       (512, 512, 1024, 3)])     # CTA pairs, several stages: the third load is withheld
def test_a_wait_that_runs_out_is_reported_and_the_next_call_is_correct(T, N, K, nth):
    qx, qw = _operands(T, N, K)
    ws = binding.alloc_workspace("cuda")
    binding.fp4q_workspace_set_wait_limit(ws, 1 << 12)
    binding.fp4q_debug_withhold_load(ws, nth)
    binding.fp4q_gemm_fwd(qx, qw, dt=binding.OUT_F32, ws=ws)        # enqueues normally: the anomaly is device-side
    torch.cuda.synchronize()                                        # the launch ends by itself, no error from the runtime
    words = ws.view(torch.int32)[:2].tolist()
    assert words[0] == FP4Q_ERR_TIMEOUT and words[1] != 0           # status, and where the kernel gave up (role and stage)
    assert binding.fp4q_workspace_status(ws) == FP4Q_ERR_TIMEOUT
    assert binding.fp4q_workspace_status(ws) == 0                   # reading the status cleared it
    # hook off, default limit: the same workspace and context serve an ordinary call
    binding.fp4q_debug_withhold_load(ws, 0)
    binding.fp4q_workspace_set_wait_limit(ws, 0)
    y = binding.fp4q_gemm_fwd(qx, qw, dt=binding.OUT_F32, ws=ws)
    torch.cuda.synchronize()
    assert binding.fp4q_workspace_status(ws) == 0
    check_gemm(y, oracle.gemm_fwd(dequant_from_gpu(qx), dequant_from_gpu(qw)), "forward after a timeout")


def test_a_small_limit_alone_does_not_disturb_a_healthy_run():
    # 2^16 polls is far more than any wait of a healthy run on this shape needs: same result, no status
    qx, qw = _operands(300, 520, 2080)
    ws = binding.alloc_workspace("cuda")
    binding.fp4q_workspace_set_wait_limit(ws, 1 << 16)
    y = binding.fp4q_gemm_fwd(qx, qw, dt=binding.OUT_F32, ws=ws)
    torch.cuda.synchronize()
    assert binding.fp4q_workspace_status(ws) == 0
    check_gemm(y, oracle.gemm_fwd(dequant_from_gpu(qx), dequant_from_gpu(qw)), "forward with a small poll limit")


def test_status_decoding_of_a_workspace_word():
    # host-side decoding: a workspace whose status word holds 7 reads as FP4Q_ERR_TIMEOUT and is cleared by the read
    ws = binding.alloc_workspace("cuda")
    ws.view(torch.int32)[0] = FP4Q_ERR_TIMEOUT
    ws.view(torch.int32)[1] = 0x300
    torch.cuda.synchronize()
    assert binding.fp4q_workspace_status(ws) == FP4Q_ERR_TIMEOUT
    assert int(ws.view(torch.int32)[0]) == 0
    assert binding.fp4q_workspace_status(ws) == 0
