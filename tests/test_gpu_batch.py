"""Parity of the batched decode entry point (one quantiser launch + one persistent weight-streaming
kernel for many independent BitLinear forwards) with the CPU oracle, element by element."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_12285_b200 import binding as bl
from paper_2504_12285_b200 import workloads as wl

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def make_case(shapes, seed, y_dtype=torch.float32, gains=False):
    """shapes: list of (M, N, K).  Returns (batch, refs) with one oracle result per problem."""
    items, refs = [], []
    for i, (M, N, K) in enumerate(shapes):
        x = wl.activations_normal(M, K, seed + 10 * i) if i % 2 == 0 else wl.activations_student_t(M, K, seed + 10 * i)
        g = wl.gain_random(K, seed + 10 * i + 1) if gains else None
        W = wl.latent_weights(N, K, seed + 10 * i + 2)
        packed, s_w = bl.bitlinear_pack_weights(W.to(DEV), wl.WEIGHT_EPS)
        wref = oracle.quantize_weights(W.numpy(), wl.WEIGHT_EPS)
        assert np.array_equal(packed.cpu().numpy(), wref["packed"])
        ref = oracle.bitlinear_forward(wl.bf16_bits(x), None if g is None else wl.bf16_bits(g), wl.RMS_EPS, wref["wq"],
                                       wref["s_w"]) if M > 0 else None
        y = torch.full((M, N), float("nan"), dtype=y_dtype, device=DEV)
        items.append((x.to(DEV), None if g is None else g.to(DEV), packed, s_w, y))
        refs.append(ref)
    return bl.ProblemBatch(items, wl.RMS_EPS), refs


def check(batch, refs):
    for (x, g, packed, s_w, y), ref in zip(batch.tensors, refs):
        if ref is None:
            continue
        ok = ref["fragile"] == 0
        assert ok.size - ok.sum() <= ok.size // 1000  # flagged rows: none at all in cases of fewer than 1000 rows
        if y.dtype == torch.float32:
            got = y.cpu().numpy().astype(np.float64)[ok]
            want = ref["y"].astype(np.float64)[ok]
            assert np.all(np.abs(got - want) <= 1e-6 * np.abs(want))
            assert np.all(got[ref["acc"][ok] == 0] == 0.0)
        else:
            want = oracle.f32_to_bf16(ref["y"]).astype(np.int32)[ok]
            got = wl.bf16_bits(y.cpu()).astype(np.int32)[ok]
            assert np.all(np.abs(got - want) <= 1)


def run(batch, reuse=False):
    ws = torch.empty(batch.workspace_bytes(), dtype=torch.uint8, device=DEV)
    bl.bitlinear_forward_batch(batch, ws, reuse_plan=False)
    if reuse:
        first = [t[4].clone() for t in batch.tensors]
        for t in batch.tensors:
            t[4].fill_(float("nan"))
        bl.bitlinear_forward_batch(batch, ws, reuse_plan=True)
        torch.cuda.synchronize()
        for a, t in zip(first, batch.tensors):
            assert torch.equal(a, t[4])
    torch.cuda.synchronize()
    assert bl.bitlinear_poll_status() == 0


def test_batch_single_token_mixed_shapes():
    shapes = [(1, 16, 256), (1, 48, 768), (1, 640, 2560), (1, 2560, 6912), (1, 128, 1024), (1, 32, 8192)]
    batch, refs = make_case(shapes, 100, gains=True)
    run(batch, reuse=True)
    check(batch, refs)


def test_batch_fewer_items_than_sms():
    batch, refs = make_case([(1, 16, 256), (1, 32, 512)], 200)
    run(batch)
    check(batch, refs)


@pytest.mark.parametrize("ms", [(2, 3, 8, 5), (16, 9, 1, 12)])
def test_batch_several_tokens(ms):
    shapes = [(ms[0], 48, 768), (ms[1], 640, 2560), (ms[2], 256, 6912), (ms[3], 128, 256)]
    batch, refs = make_case(shapes, 300 + ms[0], gains=True)
    run(batch, reuse=True)
    check(batch, refs)


@pytest.mark.parametrize("M", [2, 5, 8])
def test_batch_several_tokens_accumulators_and_shared_inputs(M):
    """2 to 8 tokens stream the weights once and multiply with int8 mma.sync: the int32 accumulators must be the oracle's
    bit for bit.  Three problems share their input (one copy in shared memory), the next has the longest row the call
    takes (eight tokens of it fill the activation arena), the last has a single token and a single row block."""
    seed = 4300 + M
    K = 2560
    x = wl.activations_student_t(M, K, seed)
    x_long = wl.activations_normal(M, 8192, seed + 1)
    x_one = wl.activations_normal(1, 512, seed + 2)
    gain = wl.gain_random(K, seed + 3)
    specs = [(x, gain, 640, K), (x, gain, 48, K), (x, gain, 2560, K), (x_long, None, 64, 8192), (x_one, None, 16, 512)]
    items, refs, accs = [], [], []
    for i, (xi, gi, N, Ki) in enumerate(specs):
        W = wl.latent_weights(N, Ki, seed + 10 + i)
        packed, s_w = bl.bitlinear_pack_weights(W.to(DEV), wl.WEIGHT_EPS)
        wref = oracle.quantize_weights(W.numpy(), wl.WEIGHT_EPS)
        refs.append(oracle.bitlinear_forward(wl.bf16_bits(xi), None if gi is None else wl.bf16_bits(gi), wl.RMS_EPS, wref["wq"], wref["s_w"]))
        y = torch.full((xi.shape[0], N), float("nan"), dtype=torch.bfloat16 if i == 1 else torch.float32, device=DEV)
        items.append((xi.to(DEV), None if gi is None else gi.to(DEV), packed, s_w, y))
        accs.append(torch.full((xi.shape[0], N), -7, dtype=torch.int32, device=DEV))
    items = [(items[0][0], items[0][1]) + it[2:] if i < 3 else it for i, it in enumerate(items)]  # one tensor for the shared input
    batch = bl.ProblemBatch(items, wl.RMS_EPS)
    ws = torch.empty(batch.workspace_bytes(), dtype=torch.uint8, device=DEV)
    bl.bitlinear_forward_batch_acc(batch, accs, ws)
    torch.cuda.synchronize()
    assert bl.bitlinear_poll_status() == 0
    for acc, ref in zip(accs, refs):
        assert not ref["fragile"].any()
        assert np.array_equal(acc.cpu().numpy(), ref["acc"])
    check(batch, refs)
    # the same bits when the quantised rows are reused
    first = [t[4].clone() for t in batch.tensors]
    for t in batch.tensors:
        t[4].fill_(float("nan"))
    bl.bitlinear_forward_batch(batch, ws, reuse_plan=True, reuse_act=True)
    torch.cuda.synchronize()
    for a, t in zip(first, batch.tensors):
        assert torch.equal(a, t[4])


@pytest.mark.parametrize("n_prob,M,order", [(6, 1, "forward"), (30, 1, "forward"), (27, 3, "forward"), (30, 1, "reversed")])
def test_batch_host_buffers_match_the_device_call(n_prob, M, order):
    """bitlinear_forward_batch_host (pinned x arena in, y arena out) against bitlinear_forward_batch on the same
    descriptors: the same bits, for a call too short to be cut into segments, for calls that are cut into three
    segments whose copies overlap the kernels, for arenas laid out against the order of the problems (not cut), and for
    a second call that reuses the plans."""
    shapes = [(48, 768), (640, 2560), (256, 1024), (128, 256), (2560, 2560), (16, 512)]
    seed = 5200 + n_prob + M
    mats = []
    for i in range(len(shapes)):
        N, K = shapes[i]
        W = wl.latent_weights(N, K, seed + i)
        mats.append(bl.bitlinear_pack_weights(W.to(DEV), wl.WEIGHT_EPS))
    specs = [shapes[i % len(shapes)] + (i % len(shapes),) for i in range(n_prob)]
    x_off, y_off, xo, yo = [], [], 0, 0
    for N, K, _ in specs:
        x_off.append(xo)
        y_off.append(yo)
        xo += (M * K * 2 + 255) // 256 * 256
        yo += (M * N * 4 + 255) // 256 * 256
    if order == "reversed":
        x_off = [xo - o - (M * K * 2 + 255) // 256 * 256 for o, (N, K, _) in zip(x_off, specs)]
        y_off = [yo - o - (M * N * 4 + 255) // 256 * 256 for o, (N, K, _) in zip(y_off, specs)]
    x_host = torch.zeros(xo, dtype=torch.uint8).pin_memory()
    y_host = torch.zeros(yo, dtype=torch.uint8).pin_memory()
    x_dev = torch.zeros(xo, dtype=torch.uint8, device=DEV)
    y_dev = torch.zeros(yo, dtype=torch.uint8, device=DEV)
    gain = {K: wl.gain_random(K, seed + 100 + K).to(DEV) for _, K in shapes}
    items = []
    for i, (N, K, mi) in enumerate(specs):
        x = wl.activations_normal(M, K, seed + 200 + i)
        nb = M * K * 2
        x_host[x_off[i]:x_off[i] + nb] = x.view(torch.uint8).reshape(-1)
        xv = x_dev[x_off[i]:x_off[i] + nb].view(torch.bfloat16).view(M, K)
        yv = y_dev[y_off[i]:y_off[i] + M * N * 4].view(torch.float32).view(M, N)
        items.append((xv, gain[K], mats[mi][0], mats[mi][1], yv))
    batch = bl.ProblemBatch(items, wl.RMS_EPS)
    ws = torch.empty(batch.workspace_bytes(), dtype=torch.uint8, device=DEV)
    # the device call on a copy of the inputs gives the expected bytes
    x_dev.copy_(x_host)
    bl.bitlinear_forward_batch(batch, ws)
    torch.cuda.synchronize()
    want = y_dev.cpu().clone()
    for reuse in (False, True):
        x_dev.zero_()
        y_dev.fill_(0xEE)
        y_host.fill_(0x11)
        bl.bitlinear_forward_batch_host(batch, x_host, x_dev, y_dev, y_host, ws, reuse_plan=reuse)  # synchronises
        assert bl.bitlinear_poll_status() == 0
        got = y_host.clone()
        # bytes between two outputs are padding of the arena: the device call left them as they were (zero), the host call
        # copies them out as they are now (0xEE); compare the outputs themselves
        for i, (N, K, _) in enumerate(specs):
            sl = slice(y_off[i], y_off[i] + M * N * 4)
            assert torch.equal(got[sl], want[sl]), (i, reuse)
        assert torch.equal(x_dev.cpu(), x_host)


def test_batch_one_workspace_serves_different_problem_lists_in_turn():
    """Calls that reuse their plan skip the host's planning when the library remembers the list it planned for that
    workspace.  Two different lists (other shapes, other token counts, the same number of problems) take turns on ONE
    workspace: every call that plans anew must replace what is remembered, every reusing call must run its own list."""
    batch_a, refs_a = make_case([(1, 48, 768), (1, 640, 2560), (1, 256, 1024), (1, 128, 256), (1, 32, 512)], 5600, gains=True)
    batch_b, refs_b = make_case([(3, 64, 512), (5, 16, 256), (2, 2560, 2560), (8, 48, 768), (1, 640, 2560)], 5700)
    ws = torch.empty(max(batch_a.workspace_bytes(), batch_b.workspace_bytes()), dtype=torch.uint8, device=DEV)
    for batch, refs in ((batch_a, refs_a), (batch_b, refs_b), (batch_a, refs_a), (batch_b, refs_b)):
        for reuse in (False, True, True):
            for t in batch.tensors:
                t[4].fill_(float("nan"))
            bl.bitlinear_forward_batch(batch, ws, reuse_plan=reuse)
            torch.cuda.synchronize()
            assert bl.bitlinear_poll_status() == 0
            check(batch, refs)


def test_batch_bf16_output_and_empty_problem():
    shapes = [(4, 64, 512), (0, 32, 256), (1, 640, 2560)]
    batch, refs = make_case(shapes, 400, y_dtype=torch.bfloat16)
    run(batch)
    check(batch, refs)


@pytest.mark.parametrize("M", [1, 4, 16])
def test_batch_one_layer_decode_step(M):
    # the seven BitLinear shapes of one 2B-style layer in a single call
    shapes = [(M, n, k) for _, n, k in wl.LAYER_SHAPES]
    batch, refs = make_case(shapes, wl.seed_for(2, 0, M))
    run(batch)
    check(batch, refs)


def test_batch_matches_single_forward_bitwise():
    shapes = [(1, n, k) for _, n, k in wl.LAYER_SHAPES[:4]]
    batch, _ = make_case(shapes, 500)
    run(batch)
    for x, g, packed, s_w, y in batch.tensors:
        y1 = bl.bitlinear_forward(x, g, packed, s_w, y.shape[1], wl.RMS_EPS)
        assert torch.equal(y, y1)


def test_batch_detects_an_overwritten_plan():
    # REUSE_PLAN trusts the workspace; if something else wrote over it, the kernels must notice and
    # compute nothing instead of following stale pointers
    batch, refs = make_case([(1, 48, 768), (2, 32, 256)], 600)
    ws = torch.empty(batch.workspace_bytes(), dtype=torch.uint8, device=DEV)
    bl.bitlinear_forward_batch(batch, ws)
    torch.cuda.synchronize()
    check(batch, refs)
    ws[:256].zero_()
    for t in batch.tensors:
        t[4].fill_(7.0)
    bl.bitlinear_forward_batch(batch, ws, reuse_plan=True)
    assert bl.bitlinear_poll_status() == 4  # workspace error, reported through the sticky status word
    for t in batch.tensors:
        assert torch.all(t[4] == 7.0)
    assert bl.bitlinear_poll_status() == 0
    bl.bitlinear_forward_batch(batch, ws)  # a fresh upload repairs it
    torch.cuda.synchronize()
    check(batch, refs)


def test_batch_many_tokens_bf16_ragged_rows_and_overwritten_plan():
    # 5 to 16 tokens: the tensor-core decode kernel; weight-row counts that are not multiples of 128,
    # one K that is a single 256-column step and one that ends in a partial ring slot (27 steps)
    shapes = [(7, 16, 256), (16, 144, 6912), (0, 32, 256), (5, 2560, 1280), (11, 272, 2560), (1, 96, 512)]
    batch, refs = make_case(shapes, 700, y_dtype=torch.bfloat16, gains=True)
    run(batch, reuse=True)
    check(batch, refs)
    ws = torch.empty(batch.workspace_bytes(), dtype=torch.uint8, device=DEV)
    bl.bitlinear_forward_batch(batch, ws)
    torch.cuda.synchronize()
    ws[:256].zero_()
    for t in batch.tensors:
        t[4].fill_(7.0)
    bl.bitlinear_forward_batch(batch, ws, reuse_plan=True)
    assert bl.bitlinear_poll_status() == 4
    for t in batch.tensors:
        assert torch.all(t[4] == 7.0)
    assert bl.bitlinear_poll_status() == 0


@pytest.mark.parametrize("M", [5, 8, 16])
def test_batch_many_tokens_match_single_forward_bitwise(M):
    shapes = [(M, n, k) for _, n, k in wl.LAYER_SHAPES[:4]]
    batch, _ = make_case(shapes, 800 + M)
    run(batch)
    for x, g, packed, s_w, y in batch.tensors:
        y1 = bl.bitlinear_forward(x, g, packed, s_w, y.shape[1], wl.RMS_EPS)
        assert torch.equal(y, y1)


@pytest.mark.parametrize("M", [1, 8, 16])  # the three kernels: one token, 2 to 8 tokens (mma.sync stream), 9 to 16 (tcgen05)
def test_batch_full_decode_step_sampled(M):
    # the launch configuration the benchmark times, with its seeded weights: 30 layers x 7 matmuls in ONE call
    # (210 problems, 521 MB of packed weights), checked on sampled outputs of every problem
    rng = np.random.default_rng(1234 + M)
    items, refs = [], []
    for layer in range(wl.N_LAYERS):
        for j, (name, n, k) in enumerate(wl.LAYER_SHAPES):
            W = wl.latent_weights(n, k, wl.layer_seed(2, layer, name))
            packed, s_w = bl.bitlinear_pack_weights(W.to(DEV), wl.WEIGHT_EPS)
            wref = oracle.quantize_weights(W.numpy(), wl.WEIGHT_EPS)
            assert np.array_equal(packed.cpu().numpy(), wref["packed"])
            n_idx = np.concatenate([rng.integers(0, n, 44), [0, n - 1, 127 % n, 128 % n]]).astype(np.int32)
            x = wl.activations_student_t(M, k, wl.seed_for(2, j, layer))
            refs.append((x, n_idx, wref["wq"][n_idx].copy(), wref["s_w"]))
            items.append((x.to(DEV), None, packed, s_w, torch.full((M, n), float("nan"), dtype=torch.float32, device=DEV)))
    batch = bl.ProblemBatch(items, wl.RMS_EPS)
    run(batch, reuse=True)
    for i, ((x, n_idx, wq_rows, s_w), (_, _, _, _, y)) in enumerate(zip(refs, batch.tensors)):
        qref = oracle.rmsnorm_quant(wl.bf16_bits(x), None, wl.RMS_EPS)
        ok_rows = np.nonzero(qref["fragile"] == 0)[0]
        y_host = y.cpu().numpy()
        assert not np.isnan(y_host).any()
        if len(ok_rows) == 0:
            continue
        m_idx = rng.choice(ok_rows, len(n_idx)).astype(np.int32)
        acc = oracle.matmul_i32_sampled(qref["q"], wq_rows, m_idx, np.arange(len(n_idx), dtype=np.int32))
        want = (oracle.dequant(acc.reshape(1, -1), s_w, np.ones(1, np.float32))[0] * qref["d"][m_idx]).astype(np.float64)
        got = y_host[m_idx, n_idx].astype(np.float64)
        assert np.all(np.abs(got - want) <= 1e-6 * np.abs(want)), i


def test_batch_many_tiny_problems_overflow_the_descriptor_cache():
    # 30,000 one-item problems of two tokens: about 203 per CTA, more than the 192 work items and the 48 descriptors
    # a CTA of the tensor-core decode kernel keeps in shared memory, so the rest is read from global memory
    N, K, M, count = 16, 256, 2, 30000
    W = wl.latent_weights(N, K, 900)
    packed, s_w = bl.bitlinear_pack_weights(W.to(DEV), wl.WEIGHT_EPS)
    wref = oracle.quantize_weights(W.numpy(), wl.WEIGHT_EPS)
    xs = wl.activations_normal(M * count, K, 901)
    xs_dev = xs.to(DEV)
    ys = torch.full((count, M, N), float("nan"), dtype=torch.float32, device=DEV)
    items = [(xs_dev[M * i:M * (i + 1)], None, packed, s_w, ys[i]) for i in range(count)]
    batch = bl.ProblemBatch(items, wl.RMS_EPS)
    run(batch)
    ref = oracle.bitlinear_forward(wl.bf16_bits(xs), None, wl.RMS_EPS, wref["wq"], wref["s_w"])  # rows are independent
    ok = ref["fragile"] == 0
    got = ys.reshape(M * count, N).cpu().numpy().astype(np.float64)[ok]
    want = ref["y"].astype(np.float64)[ok]
    assert ok.size - ok.sum() <= ok.size // 1000
    assert np.all(np.abs(got - want) <= 1e-6 * np.abs(want))


# ---- problems of more than 16 tokens in the same entry point: grouped tensor-core path ----


def test_batch_prefill_group_small_mixed_shapes():
    # ragged token counts (not multiples of the 128-row tile), several tiles along N and K, different K per problem
    shapes = [(96, 256, 512), (130, 640, 2560), (17, 128, 256), (300, 384, 768)]
    batch, refs = make_case(shapes, 700, gains=True)
    run(batch)
    check(batch, refs)


def test_batch_prefill_group_bf16_and_decode_problems_together():
    # decode-sized and prefill-sized problems in one call: each goes to its own kernel
    shapes = [(1, 640, 2560), (64, 256, 1024), (4, 48, 768), (200, 128, 512)]
    batch, refs = make_case(shapes, 800, y_dtype=torch.bfloat16)
    run(batch, reuse=True)
    check(batch, refs)


def test_batch_prefill_group_matches_single_forward_bitwise():
    shapes = [(256, 640, 2560), (256, 2560, 2560)]
    batch, _ = make_case(shapes, 900)
    run(batch)
    for x, g, packed, s_w, y in batch.tensors:
        y1 = bl.bitlinear_forward(x, g, packed, s_w, y.shape[1], wl.RMS_EPS)
        assert torch.equal(y, y1)
