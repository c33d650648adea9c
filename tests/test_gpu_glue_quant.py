"""The element-wise steps of a decoder layer fused into the quantiser launch (squared-ReLU gate, residual add,
attention stand-in; paper Section 2) against the CPU oracle: the bf16 value handed to the quantiser, the int8 codes,
scales and code sums bit for bit; the BitLinear outputs within tolerance - through the stand-alone entry point and
through all three batched paths (one token, 2 to 16 tokens, more than 16 tokens)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_12285_b200 import binding as bl
from paper_2504_12285_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def to_np(t):
    return t.detach().cpu().numpy()


def randn(m, k, seed, scale=1.0):
    return (torch.randn(m, k, generator=torch.Generator().manual_seed(seed), dtype=torch.float32) * scale).contiguous()


@pytest.mark.parametrize("M,F", [(1, 512), (5, 6912), (70, 2560), (3, 16384)])
def test_quant_act_relu2_bit_exact(M, F):
    gate, up = randn(M, F, 10 * M + 1), randn(M, F, 10 * M + 2)
    gain = wl.gain_random(F, 10 * M + 3)
    ref = oracle.relu2_rmsnorm_quant(gate.numpy(), up.numpy(), wl.bf16_bits(gain), wl.RMS_EPS)
    assert not ref["fragile"].any()
    xq, d, xsum, f = bl.bitlinear_quant_act_relu2(gate.to(DEV), up.to(DEV), gain.to(DEV), wl.RMS_EPS, want_x=True)
    assert np.array_equal(wl.bf16_bits(f.cpu()), ref["x"])
    assert np.array_equal(to_np(xq), ref["q"])
    assert np.array_equal(to_np(d), ref["d"]) and np.array_equal(to_np(xsum), ref["xsum"])
    # without the optional output, without gain
    ref = oracle.relu2_rmsnorm_quant(gate.numpy(), up.numpy(), None, wl.RMS_EPS)
    xq, d, xsum = bl.bitlinear_quant_act_relu2(gate.to(DEV), up.to(DEV), None, wl.RMS_EPS)
    assert np.array_equal(to_np(xq), ref["q"]) and np.array_equal(to_np(d), ref["d"])


def test_quant_act_relu2_all_gates_negative_is_a_zero_row():
    gate, up = -randn(2, 512, 5).abs(), randn(2, 512, 6)
    xq, d, xsum = bl.bitlinear_quant_act_relu2(gate.to(DEV), up.to(DEV), None, wl.RMS_EPS)
    assert not to_np(xq).any() and not to_np(xsum).any()
    assert np.all(to_np(d) == np.float32(1e-5) / np.float32(127.0))


def check_y(y, ref):
    ok = ref["fragile"] == 0
    assert ok.size - ok.sum() <= ok.size // 1000
    got, want = to_np(y).astype(np.float64)[ok], ref["y"].astype(np.float64)[ok]
    assert np.all(np.abs(got - want) <= 1e-6 * np.abs(want))
    assert np.all(got[ref["acc"][ok] == 0] == 0.0)


@pytest.mark.parametrize("M", [1, 4, 40, 130])  # one token, tensor-core decode, 16-token chunks, grouped GEMM
def test_batch_with_fused_steps(M):
    # a layer's dependence pattern in one call each: {q,k,v}(residual), o(stand-in), {gate,up}(residual), down(relu2)
    H, F, n_q, n_kv, hd = 512, 768, 4, 2, 128
    seed = 9000 + M
    mats = {}
    for i, (name, n, k) in enumerate((("q", H, H), ("k", n_kv * hd, H), ("v", n_kv * hd, H), ("o", H, H), ("gate", F, H),
                                      ("up", F, H), ("down", H, F))):
        W = wl.latent_weights(n, k, seed + i)
        packed, s_w = bl.bitlinear_pack_weights(W.to(DEV), wl.WEIGHT_EPS)
        mats[name] = (packed, s_w, oracle.quantize_weights(W.numpy(), wl.WEIGHT_EPS), n)
    gains = {k: wl.gain_random(k, seed + 20 + k) for k in (H, F)}
    h = wl.activations_normal(M, H, seed + 30)
    y_prev = randn(M, H, seed + 31, 0.5)
    qv, vv = randn(M, H, seed + 32), randn(M, n_kv * hd, seed + 33)
    gate, up = randn(M, F, seed + 34), randn(M, F, seed + 35)
    dev = {k: v.to(DEV) for k, v in dict(h=h, y=y_prev, q=qv, v=vv, g=gate, u=up).items()}
    gdev = {k: v.to(DEV) for k, v in gains.items()}

    def out(n):
        return torch.full((M, n), float("nan"), dtype=torch.float32, device=DEV)

    h_new = torch.zeros(M, H, dtype=torch.bfloat16, device=DEV)
    a_out = torch.zeros(M, H, dtype=torch.bfloat16, device=DEV)
    res = (bl.X_RESIDUAL, dev["y"], h_new, 0, 0)
    cases = [
        ([("q", dev["h"], res), ("k", dev["h"], res), ("v", dev["h"], res)], H,
         oracle.glue_residual(wl.bf16_bits(h), y_prev.numpy()), h_new),
        ([("o", dev["q"], (bl.X_ATTN_STANDIN, dev["v"], a_out, hd, n_q // n_kv))], H,
         oracle.glue_attn_standin(qv.numpy(), vv.numpy(), n_q, n_kv, hd), a_out),
        ([("gate", dev["h"], res), ("up", dev["h"], res)], H, oracle.glue_residual(wl.bf16_bits(h), y_prev.numpy()), h_new),
        ([("down", dev["g"], (bl.X_RELU2, dev["u"], None, 0, 0))], F, oracle.glue_relu2(gate.numpy(), up.numpy()), None),
    ]
    for probs, K, x_bits, x_out in cases:
        if x_out is not None:
            x_out.zero_()
        items = [(x, gdev[K], mats[name][0], mats[name][1], out(mats[name][3]), step) for name, x, step in probs]
        batch = bl.ProblemBatch(items, wl.RMS_EPS)
        ws = torch.empty(batch.workspace_bytes(), dtype=torch.uint8, device=DEV)
        bl.bitlinear_forward_batch(batch, ws)
        torch.cuda.synchronize()
        assert bl.bitlinear_poll_status() == 0
        if x_out is not None:
            assert np.array_equal(wl.bf16_bits(x_out.cpu()), x_bits)
        for (name, _, _), it in zip(probs, items):
            ref = oracle.bitlinear_forward(x_bits, wl.bf16_bits(gains[K]), wl.RMS_EPS, mats[name][2]["wq"], mats[name][2]["s_w"])
            check_y(it[4], ref)
        # the plan can be reused with the steps in it
        first = [it[4].clone() for it in items]
        for it in items:
            it[4].fill_(float("nan"))
        bl.bitlinear_forward_batch(batch, ws, reuse_plan=True)
        torch.cuda.synchronize()
        for a, it in zip(first, items):
            assert torch.equal(a, it[4])


def test_fused_step_equals_separate_glue_launch_bitwise():
    M, F, N = 3, 6912, 2560
    gate, up = randn(M, F, 1).to(DEV), randn(M, F, 2).to(DEV)
    W = wl.latent_weights(N, F, 3)
    packed, s_w = bl.bitlinear_pack_weights(W.to(DEV), wl.WEIGHT_EPS)
    f = torch.empty(M, F, dtype=torch.bfloat16, device=DEV)
    bl.bitlinear_glue_relu2_mul(gate, up, f)
    y_sep = bl.bitlinear_forward(f, None, packed, s_w, N, wl.RMS_EPS)
    y = torch.empty(M, N, device=DEV)
    batch = bl.ProblemBatch([(gate, None, packed, s_w, y, (bl.X_RELU2, up, None, 0, 0))], wl.RMS_EPS)
    bl.bitlinear_forward_batch(batch, torch.empty(batch.workspace_bytes(), dtype=torch.uint8, device=DEV))
    assert torch.equal(y, y_sep)


def test_fused_step_argument_checks():
    M, K, N = 2, 256, 128
    W = wl.latent_weights(N, K, 1).to(DEV)
    packed, s_w = bl.bitlinear_pack_weights(W)
    h = wl.activations_normal(M, K, 2).to(DEV)
    y2 = randn(M, K, 3).to(DEV)
    y = torch.empty(M, N, device=DEV)
    ws = torch.empty(1 << 20, dtype=torch.uint8, device=DEV)
    bad = bl.ProblemBatch([(h, None, packed, s_w, y, (bl.X_RESIDUAL, y2, h, 0, 0))], wl.RMS_EPS)  # x_out aliases x
    with pytest.raises(bl.BitLinearError) as e:
        bl.bitlinear_forward_batch(bad, ws)
    assert e.value.status == 2
    bad = bl.ProblemBatch([(y2, None, packed, s_w, y, (bl.X_ATTN_STANDIN, y2, None, 12, 1))], wl.RMS_EPS)  # head_dim % 8
    with pytest.raises(bl.BitLinearError) as e:
        bl.bitlinear_forward_batch(bad, ws)
    assert e.value.status == 2
    bad = bl.ProblemBatch([(h, None, packed, s_w, y)], wl.RMS_EPS)
    bad.array[0].x_op = 7
    with pytest.raises(bl.BitLinearError) as e:
        bl.bitlinear_forward_batch(bad, ws)
    assert e.value.status == 5
