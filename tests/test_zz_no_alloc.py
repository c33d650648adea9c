"""bitlinear_forward_static: the decode forward for callers that cannot allocate device memory.

An operator plug-in that is handed only its inputs and outputs, or a serving loop that runs after a
framework's pool has claimed the device, has no workspace to give bitlinear_forward.  The static
entry point keeps that workspace in a fixed array inside the library.  This file checks, through
the C ABI, that it returns what bitlinear_forward returns, on two calls in a row (the second call
finds the first call's leftovers in the shared array), and that sizes beyond the array are refused.
It is named so that pytest collects it after every other test file.
"""
import gc

import numpy as np
import pytest
import torch

from paper_2504_12285_b200 import binding as bl
from paper_2504_12285_b200 import workloads as wl

DEV = "cuda:0"


@pytest.mark.gpu
def test_static_forward_matches_workspace_forward_on_two_calls_in_a_row():
    # first call: 16 tokens of the widest layer input fill most of the array ...
    # second call: fewer tokens and a narrower input, so stale codes and scales sit right behind the live ones
    cases = [("down", 16, torch.float32), ("q", 3, torch.float32), ("k", 5, torch.bfloat16)]
    for i, (name, M, ydt) in enumerate(cases):
        N, K = wl.SHAPE_NK[name]
        W = wl.latent_weights(N, K, 7100 + i).to(DEV)
        packed, s_w = bl.bitlinear_pack_weights(W, wl.WEIGHT_EPS)
        x = wl.activations_normal(M, K, 7200 + i).to(DEV)
        gain = wl.gain_random(K, 7300 + i).to(DEV)
        want = bl.bitlinear_forward(x, gain, packed, s_w, N, wl.RMS_EPS, y_dtype=ydt)
        out = torch.full((M, N), float("nan"), dtype=ydt, device=DEV)  # the caller owns the output, as always
        got = None    # the previous case's output would otherwise be released inside the measured window
        gc.collect()  # nor may tensors of earlier tests that are only waiting for the collector
        torch.cuda.synchronize()
        held, free = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
        got = bl.bitlinear_forward_static(x, gain, packed, s_w, N, wl.RMS_EPS, out=out)
        torch.cuda.synchronize()
        # the call took no device memory, neither from torch's pool nor from the driver
        assert torch.cuda.memory_allocated() == held and torch.cuda.mem_get_info()[0] == free
        assert got is out
        g, w = got.float().cpu().numpy().astype(np.float64), want.float().cpu().numpy().astype(np.float64)
        assert np.all(np.isfinite(g))
        tol = 1e-6 if ydt == torch.float32 else 2.0 ** -7  # fp32: the suite's relative bound; bf16: one ulp
        assert np.all(np.abs(g - w) <= tol * np.abs(w))
        assert torch.equal(got, want)  # in fact the same kernels run: the results are identical
    assert bl.bitlinear_poll_status() == 0


def test_static_forward_refuses_sizes_beyond_its_array():
    lib = bl.lib()
    assert bl.bitlinear_static_scratch_bytes() >= 16 * 16384 + 2 * 16 * 4
    fake = 0x1000  # never dereferenced: host checks come first
    # 17 tokens do not fit
    assert lib.bitlinear_forward_static(fake, None, 1e-5, fake, fake, 17, 2560, 2560, fake, 0, None) == 4
    # an unsupported K is a shape error, a bad dtype a dtype error, a NULL pointer a NULL error
    assert lib.bitlinear_forward_static(fake, None, 1e-5, fake, fake, 1, 2560, 2500, fake, 0, None) == 2
    assert lib.bitlinear_forward_static(fake, None, 1e-5, fake, fake, 1, 2560, 2560, fake, 7, None) == 5
    assert lib.bitlinear_forward_static(None, None, 1e-5, fake, fake, 1, 2560, 2560, fake, 0, None) == 1
    assert lib.bitlinear_forward_static(fake, None, 1e-5, fake, fake, 0, 2560, 2560, fake, 0, None) == 0


@pytest.mark.gpu
def test_static_forward_binding_checks_the_output_tensor():
    N, K = 256, 512
    packed, s_w = bl.bitlinear_pack_weights(wl.latent_weights(N, K, 1).to(DEV))
    x = wl.activations_normal(2, K, 2).to(DEV)
    for bad in (torch.empty(2, N + 16, device=DEV), torch.empty(3, N, device=DEV), torch.empty(2, N),
                torch.empty(2, 2 * N, device=DEV)[:, ::2], torch.empty(2, N, dtype=torch.float16, device=DEV)):
        with pytest.raises((TypeError, ValueError)):
            bl.bitlinear_forward_static(x, None, packed, s_w, N, out=bad)
