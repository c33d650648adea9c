"""The training-time forward (master weights quantised on the fly; paper Section 2, weight quantisation bullet) against
the oracle's quantiser + forward, and against the library's own pack-then-forward route."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_12285_b200 import binding as bl
from paper_2504_12285_b200 import workloads as wl

DEV = "cuda:0"


@pytest.mark.gpu
@pytest.mark.parametrize("M,N,K,wdt", [(1, 256, 512, torch.float32), (40, 640, 2560, torch.float32), (300, 256, 768, torch.bfloat16),
                                       (5, 2560, 6912, torch.bfloat16)])
def test_master_forward_matches_oracle(M, N, K, wdt):
    W = wl.latent_weights(N, K, 6100 + M).to(wdt)
    x = wl.activations_normal(M, K, 6200 + M)
    gain = wl.gain_random(K, 6300 + M)
    ref_w = oracle.quantize_weights(W.float().numpy(), wl.WEIGHT_EPS)  # the bf16 master weights are taken exactly
    ref = oracle.bitlinear_forward(wl.bf16_bits(x), wl.bf16_bits(gain), wl.RMS_EPS, ref_w["wq"], ref_w["s_w"])
    y, packed, s_w = bl.bitlinear_forward_master(x.to(DEV), gain.to(DEV), W.to(DEV), rms_eps=wl.RMS_EPS, eps_w=wl.WEIGHT_EPS,
                                                 want_packed=True)
    torch.cuda.synchronize()
    assert bl.bitlinear_poll_status() == 0
    assert np.array_equal(packed.cpu().numpy(), ref_w["packed"])
    assert np.float32(s_w.item()) == np.float32(ref_w["s_w"])
    ok = ref["fragile"] == 0
    assert ok.size - ok.sum() <= ok.size // 1000
    got, want = y.cpu().numpy().astype(np.float64)[ok], ref["y"].astype(np.float64)[ok]
    assert np.all(np.abs(got - want) <= 1e-6 * np.abs(want))
    assert np.all(got[ref["acc"][ok] == 0] == 0.0)
    # the same bits as packing first and running the inference forward, and without the optional outputs
    y2 = bl.bitlinear_forward(x.to(DEV), gain.to(DEV), packed, s_w, N, wl.RMS_EPS)
    y3 = bl.bitlinear_forward_master(x.to(DEV), gain.to(DEV), W.to(DEV), rms_eps=wl.RMS_EPS, eps_w=wl.WEIGHT_EPS)
    assert torch.equal(y, y2) and torch.equal(y, y3)


def test_master_forward_argument_checks():
    lib = bl.lib()
    fake = 0x1000
    assert lib.bitlinear_forward_master_workspace_bytes(4, 256, 500) == 0
    need = lib.bitlinear_forward_master_workspace_bytes(4, 256, 512)
    assert need > 256 * 512 // 4
    args = (fake, None, 1e-5, fake, 0, 1e-5, 4, 256, 512, fake, 0, None, None)
    assert lib.bitlinear_forward_master(*args, fake, need - 1, None) == 4
    assert lib.bitlinear_forward_master(*args, None, need, None) == 4
    assert lib.bitlinear_forward_master(fake, None, 1e-5, None, 0, 1e-5, 4, 256, 512, fake, 0, None, None, fake, need, None) == 1
    assert lib.bitlinear_forward_master(fake, None, 1e-5, fake, 7, 1e-5, 4, 256, 512, fake, 0, None, None, fake, need, None) == 5
    assert lib.bitlinear_forward_master(fake, None, 1e-5, fake, 0, 1e-5, 4, 256, 500, fake, 0, None, None, fake, need, None) == 2
