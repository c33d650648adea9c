"""One level of a decoder layer at one token (up to four BitLinear forwards that share their input row) runs as ONE launch
that quantises the row itself.  Checked here against the CPU oracle: int32 accumulators bit for bit, outputs within the
suite's bound, the fused input steps' own outputs bit for bit - at the smallest and the largest shapes the launch takes,
with and without the promise that lets it start beside the launch in front of it, and followed by a call that reuses
its quantised row."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_12285_b200 import binding as bl
from paper_2504_12285_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def randn(m, k, seed, scale=1.0):
    return (torch.randn(m, k, generator=torch.Generator().manual_seed(seed), dtype=torch.float32) * scale).contiguous()


def make_mats(shapes, K, seed):
    mats = []
    for i, n in enumerate(shapes):
        W = wl.latent_weights(n, K, seed + i)
        packed, s_w = bl.bitlinear_pack_weights(W.to(DEV), wl.WEIGHT_EPS)
        mats.append((packed, s_w, oracle.quantize_weights(W.numpy(), wl.WEIGHT_EPS), n))
    return mats


def check(y, acc, ref):
    assert not ref["fragile"].any()
    if acc is not None:
        assert np.array_equal(acc.cpu().numpy(), ref["acc"])
    got, want = y.float().cpu().numpy().astype(np.float64), ref["y"].astype(np.float64)
    tol = 1e-6 if y.dtype == torch.float32 else 2.0 ** -7  # fp32: two roundings; bf16: one bf16 ulp on top
    assert np.all(np.abs(got - want) <= tol * np.abs(want))
    assert np.all(got[ref["acc"] == 0] == 0.0)


@pytest.mark.parametrize("K,shapes,with_gain", [
    (256, (16,), False),                         # one row block, one tile: a grid of one CTA, seven of eight warps idle
    (256, (16, 32, 48, 16), True),               # four problems, the most a level launch takes
    (2560, (2560, 640, 640), True),              # q, k, v of the 2B layer
    (2560, (6912, 6912), False),                 # gate, up: six row blocks per CTA
    (6912, (2560,), True),                       # down: 27 tiles per row block, four 16-byte vectors per thread
    (8192, (256, 16), True),                     # the largest K
])
def test_level_launch_matches_oracle(K, shapes, with_gain):
    seed = 7000 + K + len(shapes)
    mats = make_mats(shapes, K, seed)
    x = wl.activations_normal(1, K, seed + 50)
    gain = wl.gain_random(K, seed + 51) if with_gain else None
    gdev = gain.to(DEV) if with_gain else None
    ys = [torch.full((1, n), float("nan"), dtype=torch.bfloat16 if i % 2 else torch.float32, device=DEV) for i, (_, _, _, n) in enumerate(mats)]
    accs = [torch.full((1, n), -1, dtype=torch.int32, device=DEV) for (_, _, _, n) in mats]
    items = [(x.to(DEV), gdev, packed, s_w, y) for (packed, s_w, _, _), y in zip(mats, ys)]
    batch = bl.ProblemBatch(items, wl.RMS_EPS)
    ws = torch.empty(batch.workspace_bytes(), dtype=torch.uint8, device=DEV)
    refs = [oracle.bitlinear_forward(wl.bf16_bits(x), wl.bf16_bits(gain) if with_gain else None, wl.RMS_EPS, m[2]["wq"], m[2]["s_w"])
            for m in mats]
    bl.bitlinear_forward_batch_acc(batch, accs, ws)  # an ordinary launch
    torch.cuda.synchronize()
    assert bl.bitlinear_poll_status() == 0
    for y, acc, ref in zip(ys, accs, refs):
        check(y, acc, ref)
    first = [y.clone() for y in ys]
    # the same call as a programmatic dependent of whatever runs before it (here: the fills) ...
    for y in ys:
        y.fill_(float("nan"))
    bl.bitlinear_forward_batch(batch, ws, reuse_plan=True)
    torch.cuda.synchronize()
    for a, y in zip(first, ys):
        assert torch.equal(a, y)
    # ... and a call that takes the quantised row the launch left in the workspace
    for y in ys:
        y.fill_(float("nan"))
    bl.bitlinear_forward_batch(batch, ws, reuse_plan=True, reuse_act=True)
    torch.cuda.synchronize()
    for a, y in zip(first, ys):
        assert torch.equal(a, y)
    assert bl.bitlinear_poll_status() == 0


@pytest.mark.parametrize("M,K,shapes,with_gain", [
    (2, 256, (16,), False),                        # one row block, one tile
    (8, 256, (16, 32, 48, 16), True),              # four problems, eight tokens
    (3, 2560, (2560, 640, 640), True),             # q, k, v of the 2B layer
    (8, 2560, (6912, 6912), False),                # gate, up: three row blocks per CTA
    (5, 6912, (2560,), True),                      # down: 27 tiles per row block
    (8, 8192, (256, 16), True),                    # the largest K, the largest arena
    (4, 512, (16 * 700,), False),                  # several row blocks per warp
])
def test_level_launch_at_several_tokens_matches_oracle(M, K, shapes, with_gain):
    """A level at 2 to 8 tokens (a quantiser launch and the multi-token stream kernel on a handful of problems that share
    their input): int32 accumulators bit for bit, outputs within the suite's bound, the same bits with the plan and then
    the quantised rows reused."""
    seed = 7300 + K + len(shapes) + M
    mats = make_mats(shapes, K, seed)
    x = wl.activations_student_t(M, K, seed + 50)
    gain = wl.gain_random(K, seed + 51) if with_gain else None
    gdev = gain.to(DEV) if with_gain else None
    ys = [torch.full((M, n), float("nan"), dtype=torch.bfloat16 if i % 2 else torch.float32, device=DEV) for i, (_, _, _, n) in enumerate(mats)]
    accs = [torch.full((M, n), -1, dtype=torch.int32, device=DEV) for (_, _, _, n) in mats]
    xd = x.to(DEV)
    items = [(xd, gdev, packed, s_w, y) for (packed, s_w, _, _), y in zip(mats, ys)]
    batch = bl.ProblemBatch(items, wl.RMS_EPS)
    ws = torch.empty(batch.workspace_bytes(), dtype=torch.uint8, device=DEV)
    refs = [oracle.bitlinear_forward(wl.bf16_bits(x), wl.bf16_bits(gain) if with_gain else None, wl.RMS_EPS, m[2]["wq"], m[2]["s_w"])
            for m in mats]
    bl.bitlinear_forward_batch_acc(batch, accs, ws)
    torch.cuda.synchronize()
    assert bl.bitlinear_poll_status() == 0
    for y, acc, ref in zip(ys, accs, refs):
        ok = ref["fragile"] == 0
        assert ok.all()
        assert np.array_equal(acc.cpu().numpy(), ref["acc"])
        got, want = y.float().cpu().numpy().astype(np.float64), ref["y"].astype(np.float64)
        tol = 1e-6 if y.dtype == torch.float32 else 2.0 ** -7
        assert np.all(np.abs(got - want) <= tol * np.abs(want))
    first = [y.clone() for y in ys]
    for kwargs in (dict(reuse_plan=True), dict(reuse_plan=True, reuse_act=True)):
        for y in ys:
            y.fill_(float("nan"))
        bl.bitlinear_forward_batch(batch, ws, **kwargs)
        torch.cuda.synchronize()
        for a, y in zip(first, ys):
            assert torch.equal(a, y)
    assert bl.bitlinear_poll_status() == 0


def test_level_launch_with_fused_steps_writes_their_output_once():
    H, F, n_q, n_kv, hd = 2560, 6912, 20, 5, 128
    seed = 7700
    (pd, sd, rd, _), = make_mats((H,), F, seed)
    (pg, sg, rg, _), (pu, su, ru, _) = make_mats((F, F), H, seed + 10)
    (po, so, ro, _), = make_mats((H,), H, seed + 20)
    gain_f, gain_h = wl.gain_random(F, seed + 30), wl.gain_random(H, seed + 31)
    h = wl.activations_normal(1, H, seed + 40)
    y_prev, gate, up = randn(1, H, seed + 41, 0.5), randn(1, F, seed + 42), randn(1, F, seed + 43)
    qv, vv = randn(1, H, seed + 44), randn(1, n_kv * hd, seed + 45)

    def run(items, K):
        batch = bl.ProblemBatch(items, wl.RMS_EPS)
        ws = torch.empty(batch.workspace_bytes(), dtype=torch.uint8, device=DEV)
        bl.bitlinear_forward_batch(batch, ws)
        torch.cuda.synchronize()
        assert bl.bitlinear_poll_status() == 0

    # residual in front of gate / up: the new hidden state is an output of the launch
    h_new = torch.zeros(1, H, dtype=torch.bfloat16, device=DEV)
    yg, yu = torch.empty(1, F, device=DEV), torch.empty(1, F, device=DEV)
    step = (bl.X_RESIDUAL, y_prev.to(DEV), h_new, 0, 0)
    run([(h.to(DEV), gain_h.to(DEV), pg, sg, yg, step), (h.to(DEV), gain_h.to(DEV), pu, su, yu, step)], H)
    x_bits = oracle.glue_residual(wl.bf16_bits(h), y_prev.numpy())
    assert np.array_equal(wl.bf16_bits(h_new.cpu()), x_bits)
    check(yg, None, oracle.bitlinear_forward(x_bits, wl.bf16_bits(gain_h), wl.RMS_EPS, rg["wq"], rg["s_w"]))
    check(yu, None, oracle.bitlinear_forward(x_bits, wl.bf16_bits(gain_h), wl.RMS_EPS, ru["wq"], ru["s_w"]))
    # squared-ReLU gate in front of down (two fp32 vectors of 6912 elements per CTA)
    yd = torch.empty(1, H, device=DEV)
    run([(gate.to(DEV), gain_f.to(DEV), pd, sd, yd, (bl.X_RELU2, up.to(DEV), None, 0, 0))], F)
    check(yd, None, oracle.bitlinear_forward(oracle.glue_relu2(gate.numpy(), up.numpy()), wl.bf16_bits(gain_f), wl.RMS_EPS, rd["wq"], rd["s_w"]))
    # attention stand-in in front of o
    a_out = torch.zeros(1, H, dtype=torch.bfloat16, device=DEV)
    yo = torch.empty(1, H, device=DEV)
    run([(qv.to(DEV), gain_h.to(DEV), po, so, yo, (bl.X_ATTN_STANDIN, vv.to(DEV), a_out, hd, n_q // n_kv))], H)
    a_bits = oracle.glue_attn_standin(qv.numpy(), vv.numpy(), n_q, n_kv, hd)
    assert np.array_equal(wl.bf16_bits(a_out.cpu()), a_bits)
    check(yo, None, oracle.bitlinear_forward(a_bits, wl.bf16_bits(gain_h), wl.RMS_EPS, ro["wq"], ro["s_w"]))


def test_single_forward_at_one_token_equals_the_two_launch_route():
    # bitlinear_forward at one token is one launch; quantising and multiplying in two calls must give the same bits
    N, K = 2560, 6912
    W = wl.latent_weights(N, K, 7800)
    packed, s_w = bl.bitlinear_pack_weights(W.to(DEV), wl.WEIGHT_EPS)
    x, gain = wl.activations_normal(1, K, 7801).to(DEV), wl.gain_random(K, 7802).to(DEV)
    y1 = bl.bitlinear_forward(x, gain, packed, s_w, N, wl.RMS_EPS)
    xq, d, xsum = bl.bitlinear_quant_act(x, gain, wl.RMS_EPS)
    y2 = bl.bitlinear_matmul_q(xq, d, xsum, packed, s_w, N)
    assert torch.equal(y1, y2)
