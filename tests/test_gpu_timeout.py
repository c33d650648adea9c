"""The bounded device-side waits: a wait that runs out must end the kernel by itself, leave the context usable and
show up exactly once in bitlinear_poll_status.  The self-test kernel waits on a barrier that nothing ever arrives on,
with a limit of a millisecond; no production kernel is involved and nothing is left waiting."""
import time

import numpy as np
import pytest
import torch

import oracle
from paper_2504_12285_b200 import binding as bl
from paper_2504_12285_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_wait_that_runs_out_reports_timeout_once_and_the_library_keeps_working():
    assert bl.bitlinear_poll_status() == 0
    t0 = time.perf_counter()
    bl.bitlinear_selftest_wait_timeout(1000)  # 1 ms
    torch.cuda.synchronize()                  # the kernel returns by itself
    assert time.perf_counter() - t0 < 5.0
    assert bl.bitlinear_poll_status() == 8    # BITLINEAR_ERR_TIMEOUT, read and cleared
    assert bl.bitlinear_poll_status() == 0
    assert bl.status_string(8) == "device-side wait timed out"
    # a normal call afterwards is bit-correct
    N, K, M = 256, 512, 3
    W = wl.latent_weights(N, K, 71)
    packed, s_w = bl.bitlinear_pack_weights(W.to(DEV), wl.WEIGHT_EPS)
    ref_w = oracle.quantize_weights(W.numpy(), wl.WEIGHT_EPS)
    x = wl.activations_normal(M, K, 72)
    xq, d, xsum = bl.bitlinear_quant_act(x.to(DEV), None, wl.RMS_EPS)
    y, acc = bl.bitlinear_matmul_q(xq, d, xsum, packed, s_w, N, want_acc=True)
    ref = oracle.bitlinear_forward(wl.bf16_bits(x), None, wl.RMS_EPS, ref_w["wq"], ref_w["s_w"])
    assert not ref["fragile"].any()
    assert np.array_equal(acc.cpu().numpy(), ref["acc"])
    assert bl.bitlinear_poll_status() == 0


def test_selftest_rejects_limits_outside_its_range():
    for bad in (0, 100001):
        with pytest.raises(bl.BitLinearError) as e:
            bl.bitlinear_selftest_wait_timeout(bad)
        assert e.value.status == 2
