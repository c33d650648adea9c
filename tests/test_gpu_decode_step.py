"""The parts of a decode step that are not BitLinear (rotary embedding + cache append, grouped-query decode attention,
output head, embedding) against the fp64 oracle.  These are floating-point kernels whose summation order differs from
the oracle's, so the bounds are tolerances, derived below from the arithmetic."""
import numpy as np
import pytest
import torch

import oracle
from oracle import decode_step as ds
from paper_2504_12285_b200 import binding as bl
from paper_2504_12285_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def bits(t):
    return wl.bf16_bits(t.cpu())


def bf(a):
    return oracle.bf16_to_f32(a).astype(np.float64)


def cache_to_dev(t, n_kv, hd):
    """[n_seq, t_max, n_kv * hd] (one row per position, as the oracle reads it) -> the library's [n_seq, n_kv, t_max, hd]."""
    n_seq, t_max, _ = t.shape
    return t.view(n_seq, t_max, n_kv, hd).permute(0, 2, 1, 3).contiguous().to(DEV)


def cache_bits(c):
    """The library's [n_seq, n_kv, t_max, hd] cache -> bf16 bit patterns [n_seq, t_max, n_kv * hd]."""
    n_seq, n_kv, t_max, hd = c.shape
    return bits(c.permute(0, 2, 1, 3).reshape(n_seq, t_max, n_kv * hd).contiguous())


def randn(shape, seed, scale=1.0):
    return (torch.randn(*shape, generator=torch.Generator().manual_seed(seed), dtype=torch.float32) * scale).contiguous()


@pytest.mark.parametrize("M,n_q,n_kv,hd", [(1, 20, 5, 128), (7, 4, 2, 64), (16, 20, 5, 128)])
def test_rope_and_cache_append(M, n_q, n_kv, hd):
    t_max, n_seq = 4096, 3
    q, k, v = randn((M, n_q * hd), 1), randn((M, n_kv * hd), 2), randn((M, n_kv * hd), 3)
    rng = np.random.default_rng(M)
    pos = rng.choice(t_max, M, replace=False).astype(np.int32)  # distinct rows, up to the end of the cache
    pos[0] = 0
    seq = rng.integers(0, n_seq, M).astype(np.int32)
    kc = torch.zeros(n_seq, n_kv, t_max, hd, dtype=torch.bfloat16, device=DEV)
    vc = torch.zeros_like(kc)
    q_out = bl.bitlinear_rope_kv(q.to(DEV), k.to(DEV), v.to(DEV), torch.from_numpy(pos).to(DEV), kc, vc, n_q, n_kv, hd,
                                 seq_ids=torch.from_numpy(seq).to(DEV))
    torch.cuda.synchronize()
    q_ref = ds.rope(q.numpy(), pos, n_q, hd)
    k_ref = ds.rope(k.numpy(), pos, n_kv, hd)
    # the kernel forms the angle in fp64 and rotates in fp32 (error below 2^-22 of the pair's norm), then rounds to bf16:
    # one bf16 ulp of the result (2^-8 relative after rounding) plus that absolute slack
    def close(got_bits, ref, norm):
        got = bf(got_bits)
        assert np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 2.0 ** -20 * norm)

    def pair_norm(x, nh):  # the norm of the (i, i + hd/2) pair each coordinate belongs to
        xs = x.astype(np.float64).reshape(-1, nh, 2, hd // 2)
        return np.broadcast_to(np.sqrt((xs ** 2).sum(2, keepdims=True)), xs.shape).reshape(x.shape[0], -1)

    close(bits(q_out), q_ref, pair_norm(q.numpy(), n_q))
    assert np.array_equal(bits(q_out)[0], oracle.f32_to_bf16(q.numpy()[0]))  # position 0: the identity, bit for bit
    kc_h, vc_h = cache_bits(kc), cache_bits(vc)
    for m in range(M):
        close(kc_h[seq[m], pos[m]][None], k_ref[m][None], pair_norm(k.numpy(), n_kv)[m][None])
        assert np.array_equal(vc_h[seq[m], pos[m]], oracle.f32_to_bf16(v.numpy()[m]))  # values are stored unrotated
    # nothing else was written
    mask = np.ones((n_seq, t_max), bool)
    mask[seq, pos] = False
    assert not kc_h[mask].any() and not vc_h[mask].any()


@pytest.mark.parametrize("n_q,n_kv,hd,lengths", [
    (20, 5, 128, [4096]),                      # the 2B configuration at a full cache: 64 slices
    (20, 5, 128, [1, 7, 8, 9, 300, 1000]),     # ragged lengths, several tokens
    (4, 2, 64, [5, 64, 65, 513]),
    (8, 1, 128, [33]),                         # eight query heads on one KV head
])
def test_attention_decode(n_q, n_kv, hd, lengths):
    M = len(lengths)
    t_max = max(max(lengths), 16)
    n_seq = 2
    kc = randn((n_seq, t_max, n_kv * hd), 10).to(torch.bfloat16)
    vc = randn((n_seq, t_max, n_kv * hd), 11).to(torch.bfloat16)
    q = randn((M, n_q * hd), 12, 2.0).to(torch.bfloat16)  # scores with a standard deviation of about 2: a peaked softmax
    seq = (np.arange(M) % n_seq).astype(np.int32)
    out = bl.bitlinear_attention_decode(q.to(DEV), cache_to_dev(kc, n_kv, hd), cache_to_dev(vc, n_kv, hd),
                                        torch.tensor(lengths, dtype=torch.int32, device=DEV),
                                        n_q, n_kv, hd, seq_ids=torch.from_numpy(seq).to(DEV))
    torch.cuda.synchronize()
    got = bf(bits(out))
    kb, vb, qb = bits(kc), bits(vc), bits(q)
    for m in range(M):
        ref = ds.attention_decode(qb[m], kb[seq[m]], vb[seq[m]], lengths[m], n_q, n_kv, hd)
        # fp32 scores (error ~1e-6 relative to |q||k|), fp32 softmax and accumulation, one bf16 rounding at the end:
        # 2^-8 relative for the rounding plus 1e-4 of the largest value magnitude for the fp32 arithmetic
        vmax = np.abs(bf(vb[seq[m], :lengths[m]])).max()
        assert np.all(np.abs(got[m] - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-4 * vmax), m


@pytest.mark.parametrize("n_q,n_kv,hd,lengths", [
    (20, 5, 128, [4096]),                          # the newest row is the last row of a full cache
    (20, 5, 128, [1, 7, 16, 17, 64, 65, 300, 1000, 0, 1001, 5]),  # every warp and tile boundary; two lengths that are no token
    (4, 2, 64, [5, 64, 65, 513, 48]),
    (8, 1, 128, [33]),
])
def test_attention_with_append_equals_the_two_call_route(n_q, n_kv, hd, lengths):
    """Rotary embedding + cache append done inside the attention launches: the caches and the result must carry the bits
    of bitlinear_rope_kv followed by bitlinear_attention_decode, and the result is checked against the oracle."""
    M = len(lengths)
    t_max = max(min(max(lengths), 4096), 16) if max(lengths) != 1001 else 1000
    n_seq = M + 1
    q, k, v = randn((M, n_q * hd), 30, 2.0), randn((M, n_kv * hd), 31), randn((M, n_kv * hd), 32)
    kc0 = cache_to_dev(randn((n_seq, t_max, n_kv * hd), 33).to(torch.bfloat16), n_kv, hd)
    vc0 = cache_to_dev(randn((n_seq, t_max, n_kv * hd), 34).to(torch.bfloat16), n_kv, hd)
    seq = np.arange(M, dtype=np.int32)[::-1].copy()  # distinct sequences
    if M > 4:
        seq[4] = n_seq + 3  # a sequence that does not exist: nothing stored, a zero row
    live = [m for m in range(M) if 1 <= lengths[m] <= t_max and seq[m] < n_seq]
    len_d = torch.tensor(lengths, dtype=torch.int32, device=DEV)
    seq_d = torch.from_numpy(seq).to(DEV)
    table = bl.bitlinear_rope_table(hd, t_max + 5, device=DEV)  # a table longer than the cache is fine
    # the two-call route
    kc_a, vc_a = kc0.clone(), vc0.clone()
    q_rot = bl.bitlinear_rope_kv(q.to(DEV), k.to(DEV), v.to(DEV), len_d - 1, kc_a, vc_a, n_q, n_kv, hd, seq_ids=seq_d)
    out_a = bl.bitlinear_attention_decode(q_rot, kc_a, vc_a, len_d, n_q, n_kv, hd, seq_ids=seq_d)
    # one call
    kc_b, vc_b = kc0.clone(), vc0.clone()
    out_b = bl.bitlinear_attention_decode_append(q.to(DEV), k.to(DEV), v.to(DEV), table, kc_b, vc_b, len_d, n_q, n_kv, hd, seq_ids=seq_d)
    torch.cuda.synchronize()
    assert bl.bitlinear_poll_status() == 0
    assert torch.equal(kc_a, kc_b) and torch.equal(vc_a, vc_b)
    changed = (kc_b != kc0).any(dim=-1).sum().item()
    assert changed <= len(live) * n_kv and (not live or changed > 0)
    for m in range(M):
        if m in live:
            assert torch.equal(out_a[m], out_b[m]), m
        else:
            assert not out_b[m].any(), m  # a length of t_max + 1 is clamped by the plain call, no token for this one
    got, kb, vb, qb = bf(bits(out_b)), cache_bits(kc_b), cache_bits(vc_b), bits(q_rot)
    for m in live:
        ref = ds.attention_decode(qb[m], kb[seq[m]], vb[seq[m]], lengths[m], n_q, n_kv, hd)
        vmax = np.abs(bf(vb[seq[m], :lengths[m]])).max()
        assert np.all(np.abs(got[m] - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-4 * vmax), m


def test_attention_hand_cases():
    n_q, n_kv, hd, T = 4, 2, 64, 40
    kc = randn((1, T, n_kv * hd), 20).to(torch.bfloat16)
    vc = randn((1, T, n_kv * hd), 21).to(torch.bfloat16)
    lengths = torch.tensor([1, 25], dtype=torch.int32, device=DEV)
    q = torch.zeros(2, n_q * hd, dtype=torch.bfloat16)
    q[0] = randn((n_q * hd,), 22).to(torch.bfloat16)
    out = bf(bits(bl.bitlinear_attention_decode(q.to(DEV), cache_to_dev(kc, n_kv, hd), cache_to_dev(vc, n_kv, hd), lengths,
                                                n_q, n_kv, hd)))
    v64 = bf(bits(vc))[0].reshape(T, n_kv, hd)
    # length 1: the first value row, whatever the query (exact: the weight is 1)
    assert np.array_equal(out[0].reshape(n_q, hd)[3], v64[0, 1])
    # zero query: the mean of the first 25 value rows
    want = v64[:25].mean(axis=0)
    assert np.all(np.abs(out[1].reshape(n_q, hd)[0] - want[0]) <= 2.0 ** -8 * np.abs(want[0]) + 1e-5)


@pytest.mark.parametrize("M,V,K", [(1, 1000, 256), (3, 5000, 2560), (5, 1003, 264), (8, 777, 2560), (16, 2048, 2560), (1, 128256, 2560),
                                   (16, 128256, 2560)])
def test_lm_head(M, V, K):
    x = randn((M, K), 30).to(torch.bfloat16)
    table = randn((V, K), 31, 0.05).to(torch.bfloat16)
    logits = bl.bitlinear_lm_head(x.to(DEV), table.to(DEV)).cpu().numpy().astype(np.float64)
    if V > 20000:  # the full vocabulary: sampled rows
        rows = np.concatenate([np.random.default_rng(1).integers(0, V, 2000), [0, V - 1]])
    else:
        rows = np.arange(V)
    ref = ds.lm_head(bits(x), bits(table)[rows])
    # K products of bf16 values accumulated in fp32 in another order: error below K * 2^-24 * sum |x e|
    bound = K * 2.0 ** -24 * (np.abs(bf(bits(x))) @ np.abs(bf(bits(table)[rows])).T)
    assert np.all(np.abs(logits[:, rows] - ref) <= bound + 1e-30)
    assert not np.isnan(logits).any()


def test_embed():
    V, K = 300, 512
    table = randn((V, K), 40).to(torch.bfloat16)
    ids = torch.tensor([0, 299, 17, 17, 5], dtype=torch.int32)
    out = bl.bitlinear_embed(ids.to(DEV), table.to(DEV))
    assert np.array_equal(bits(out), ds.embed(ids.numpy(), bits(table)))


def test_argument_checks():
    lib = bl.lib()
    fake = 0x1000
    assert lib.bitlinear_lm_head(fake, fake, 17, 100, 256, fake, None) == 2
    assert lib.bitlinear_lm_head(fake, fake, 1, 100, 250, fake, None) == 2
    assert lib.bitlinear_lm_head(None, fake, 1, 100, 256, fake, None) == 1
    assert lib.bitlinear_attention_workspace_bytes(1, 20, 5, 96, 128) == 0  # head_dim 64 or 128
    assert lib.bitlinear_attention_decode(fake, fake, fake, fake, None, 1, 20, 6, 128, 1, 128, fake, fake, 1 << 20, None) == 2
    assert lib.bitlinear_attention_decode(fake, fake, fake, fake, None, 1, 20, 5, 128, 0, 128, fake, fake, 1 << 20, None) == 2
    assert lib.bitlinear_attention_decode(fake, fake, fake, fake, None, 1, 20, 5, 128, 1, 128, fake, fake, 16, None) == 4
    assert lib.bitlinear_rope_kv(fake, fake, fake, fake, None, 1, 20, 5, 100, 500000.0, fake, fake, fake, 1, 16, None) == 2
    assert lib.bitlinear_embed(fake, fake, 0, 10, 256, fake, None) == 0


@pytest.mark.parametrize("append_in_attention", [False, True])
def test_whole_decode_step_stage_by_stage(append_in_attention):
    """One decoder layer + embedding + output head through DecodeStep; every stage is checked against the oracle applied
    to the values the GPU fed into that stage (a quantiser between two stages would turn a last-bit difference of an
    earlier floating-point stage into a different code, so the stages are not chained on the oracle side)."""
    from paper_2504_12285_b200 import chain as gpu_chain

    H, F, n_q, n_kv, hd, V, M, t_max = 256, 512, 4, 2, 64, 500, 3, 80
    kv = n_kv * hd
    mats, layer = {}, {}
    for i, (name, n, k) in enumerate((("q", H, H), ("k", kv, H), ("v", kv, H), ("o", H, H), ("gate", F, H), ("up", F, H),
                                      ("down", H, F))):
        W = wl.latent_weights(n, k, 8100 + i)
        packed, s_w = bl.bitlinear_pack_weights(W.to(DEV), wl.WEIGHT_EPS)
        gain = wl.gain_random(k, 8200 + i)
        layer[name] = (packed, s_w, gain.to(DEV))
        mats[name] = (oracle.quantize_weights(W.numpy(), wl.WEIGHT_EPS), wl.bf16_bits(gain))
    table = randn((V, H), 50).to(torch.bfloat16)
    st = gpu_chain.DecodeStep([layer], table.to(DEV), M, t_max, H, F, n_q, n_kv, hd, wl.RMS_EPS, device=DEV,
                              append_in_attention=append_in_attention)
    assert st.launches_per_layer == (10 if append_in_attention else 11)
    # a context in the caches: sequence m has positions[m] earlier tokens
    pos = np.array([0, 37, 79], np.int32)
    st.k_cache[0].copy_(cache_to_dev(randn((M, t_max, kv), 51).to(torch.bfloat16), n_kv, hd))
    st.v_cache[0].copy_(cache_to_dev(randn((M, t_max, kv), 52).to(torch.bfloat16), n_kv, hd))
    st.set_positions(torch.from_numpy(pos).to(DEV))
    ids = torch.tensor([7, 499, 123], dtype=torch.int32)
    logits = st.step(ids.to(DEV))
    torch.cuda.synchronize()
    assert bl.bitlinear_poll_status() == 0

    def bitlinear(name, x_bits):
        ref = oracle.bitlinear_forward(x_bits, mats[name][1], wl.RMS_EPS, mats[name][0]["wq"], mats[name][0]["s_w"])
        assert not ref["fragile"].any()
        return ref["y"].astype(np.float64)

    def close_f32(got, want):
        assert np.all(np.abs(got.cpu().numpy().astype(np.float64) - want) <= 1e-6 * np.abs(want))

    h0 = ds.embed(ids.numpy(), bits(table))
    assert np.array_equal(bits(st.h_in), h0)
    for name, buf in (("q", st.q), ("k", st.k), ("v", st.v)):
        close_f32(buf, bitlinear(name, h0))
    qg, kg, vg = (t.cpu().numpy() for t in (st.q, st.k, st.v))
    q_ref, k_ref = ds.rope(qg, pos, n_q, hd), ds.rope(kg, pos, n_kv, hd)
    slack = 2.0 ** -20 * max(np.abs(qg).max(), np.abs(kg).max()) * 2
    if append_in_attention:  # the rotated q stays in registers: take it from the rotary launch (same bits, tested above)
        scratch = torch.zeros_like(st.k_cache[0]), torch.zeros_like(st.v_cache[0])
        st.q_rot = bl.bitlinear_rope_kv(st.q, st.k, st.v, st.positions, *scratch, n_q, n_kv, hd, seq_ids=st.seq_ids)
    assert np.all(np.abs(bf(bits(st.q_rot)) - q_ref) <= 2.0 ** -8 * np.abs(q_ref) + slack)
    kc, vc = cache_bits(st.k_cache[0]), cache_bits(st.v_cache[0])
    for m in range(M):
        assert np.all(np.abs(bf(kc[m, pos[m]]) - k_ref[m]) <= 2.0 ** -8 * np.abs(k_ref[m]) + slack)
        assert np.array_equal(vc[m, pos[m]], oracle.f32_to_bf16(vg[m]))
        a_ref = ds.attention_decode(bits(st.q_rot)[m], kc[m], vc[m], int(pos[m]) + 1, n_q, n_kv, hd)
        vmax = np.abs(bf(vc[m, :pos[m] + 1])).max()
        assert np.all(np.abs(bf(bits(st.attn))[m] - a_ref) <= 2.0 ** -8 * np.abs(a_ref) + 1e-4 * vmax)
    close_f32(st.o, bitlinear("o", bits(st.attn)))
    h_mid = oracle.glue_residual(h0, st.o.cpu().numpy())
    close_f32(st.g, bitlinear("gate", h_mid))
    close_f32(st.u, bitlinear("up", h_mid))
    close_f32(st.dn, bitlinear("down", oracle.glue_relu2(st.g.cpu().numpy(), st.u.cpu().numpy())))
    h_end = oracle.glue_residual(h_mid, st.dn.cpu().numpy())
    assert np.array_equal(bits(st.h_mid), h_end)
    ref = ds.lm_head(h_end, bits(table))
    bound = H * 2.0 ** -24 * (np.abs(bf(h_end)) @ np.abs(bf(bits(table))).T)
    assert np.all(np.abs(logits.cpu().numpy().astype(np.float64) - ref) <= bound)


def test_recorded_step_replays_with_new_tokens_and_positions():
    """DecodeStep.capture(): one recording, replayed for two consecutive tokens, gives what the eager calls give."""
    from paper_2504_12285_b200 import chain as gpu_chain

    H, F, n_q, n_kv, hd, V, M, t_max = 256, 512, 4, 2, 64, 300, 2, 64
    layers = []
    for li in range(2):
        layer = {}
        for i, (name, n, k) in enumerate((("q", H, H), ("k", n_kv * hd, H), ("v", n_kv * hd, H), ("o", H, H), ("gate", F, H),
                                          ("up", F, H), ("down", H, F))):
            packed, s_w = bl.bitlinear_pack_weights(wl.latent_weights(n, k, 8300 + 10 * li + i).to(DEV), wl.WEIGHT_EPS)
            layer[name] = (packed, s_w, None)
        layers.append(layer)
    table = randn((V, H), 60).to(torch.bfloat16).to(DEV)

    def run(recorded):
        st = gpu_chain.DecodeStep(layers, table, M, t_max, H, F, n_q, n_kv, hd, wl.RMS_EPS, device=DEV)
        if recorded:
            st.capture()
            for c in st.k_cache + st.v_cache:
                c.zero_()  # the recording's own runs appended rows at position 0
        outs = []
        for t, ids in enumerate(([3, 7], [11, 299])):
            st.set_positions(torch.full((M,), t, dtype=torch.int32, device=DEV))
            idt = torch.tensor(ids, dtype=torch.int32, device=DEV)
            if recorded:
                st.ids_buf.copy_(idt)
                outs.append(st.step_graph().clone())
            else:
                outs.append(st.step(idt).clone())
        torch.cuda.synchronize()
        return outs

    eager, replayed = run(False), run(True)
    for a, b in zip(eager, replayed):
        assert torch.isfinite(a).all() and torch.equal(a, b)
    assert bl.bitlinear_poll_status() == 0


def test_replayed_token_is_deterministic_at_full_layer_shapes():
    """Every launch of a recorded token is a programmatic dependent of the one before it and starts early (weights, gains
    and scales are fetched while the predecessor still runs).  A read that came too early would show as a result that
    changes from replay to replay: 300 replays of one token on two full-size layers must give the same bits, and the
    same bits as the eager calls."""
    from paper_2504_12285_b200 import chain as gpu_chain

    H, F, n_q, n_kv, hd, V, t_max = wl.HIDDEN, wl.FFN, wl.N_Q_HEADS, wl.N_KV_HEADS, wl.HEAD_DIM, 4096, 4096
    layers = []
    for li in range(2):
        layer = {}
        for i, (name, n, k) in enumerate(wl.LAYER_SHAPES):
            packed, s_w = bl.bitlinear_pack_weights(wl.latent_weights(n, k, 8500 + 10 * li + i).to(DEV), wl.WEIGHT_EPS)
            layer[name] = (packed, s_w, wl.gain_random(k, 8600 + 10 * li + i).to(DEV))
        layers.append(layer)
    table = randn((V, H), 70, 0.05).to(torch.bfloat16).to(DEV)
    st = gpu_chain.DecodeStep(layers, table, 1, t_max, H, F, n_q, n_kv, hd, wl.RMS_EPS, device=DEV)
    gen = torch.Generator(device=DEV).manual_seed(71)
    for c in st.k_cache + st.v_cache:
        c.copy_(torch.randn(c.shape, generator=gen, device=DEV))
    st.set_positions(torch.tensor([t_max - 1], dtype=torch.int32, device=DEV))
    ids = torch.tensor([1234], dtype=torch.int32, device=DEV)
    want = st.step(ids).clone()
    assert torch.isfinite(want).all()
    st.capture()
    st.ids_buf.copy_(ids)
    for _ in range(300):
        got = st.step_graph()
        assert torch.equal(got, want)  # (the comparison synchronises: replays do not pile up)
    for _ in range(50):  # and back to back: the first launch of a token overlaps the last launches of the token before
        st.step_graph()
    assert torch.equal(st.logits, want)
    assert bl.bitlinear_poll_status() == 0
