"""Failure detection without a fault: a bounded device-side wait is made to run out (a barrier nobody arrives at, a
limit of a few milliseconds), the kernel returns by itself, the host reads NVFP4_ERR_TIMEOUT and the recorded code
from the status word, the word is cleared, and the device goes on working."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import parity as P
from paper_2509_25149_b200 import binding as B
from paper_2509_25149_b200 import synth

pytestmark = pytest.mark.gpu
ERR_TIMEOUT, ERR_ARG = 7, 4


def test_expired_wait_is_reported_and_the_device_stays_usable():
    L = B.lib()
    B.nvfp4_device_status()  # clean before
    assert L.nvfp4_test_wait_timeout(0, None) == ERR_ARG and L.nvfp4_test_wait_timeout(10 ** 9, None) == ERR_ARG
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    B.nvfp4_test_wait_timeout(3_000_000)  # 3 ms
    t1.record()
    detail = ctypes.c_uint32(0)
    assert L.nvfp4_device_status(None, ctypes.byref(detail)) == ERR_TIMEOUT
    assert detail.value == 0x7E570001
    assert 2.5 <= t0.elapsed_time(t1) <= 200.0  # it waited out its limit and came back by itself
    with pytest.raises(B.NVFP4Error):
        B.nvfp4_test_wait_timeout(2_000_000)
        B.nvfp4_device_status()
    B.nvfp4_device_status()  # reading cleared the word

    # a normal quantize + GEMM right after it: parity as usual
    a = synth.normal_bf16((256, 512), 1.0, 21)
    b = synth.normal_bf16((256, 512), 0.02, 22)
    A, _ = P.gpu_quantize(a)
    Bq, _ = P.gpu_quantize(b, block_rows=16)
    D = torch.empty((256, 256), dtype=torch.bfloat16, device="cuda")
    B.nvfp4_gemm(A, Bq, D)
    B.nvfp4_device_status()
    Dref, T = P.gemm_reference(oracle.quantize(synth.bits(a)), oracle.quantize(synth.bits(b), block_rows=16))
    P.assert_gemm_close(D.float().cpu().numpy(), Dref, T, True, "GEMM after an expired wait")
