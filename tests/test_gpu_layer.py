"""GPU parity of the layer pieces (linear, RMSNorm, rotary embedding of the block, SwiGLU) with the oracle."""
import numpy as np
import pytest
import torch

import paper_2509_24007_b200 as pk
from paper_2509_24007_b200.harness import DeviceProblem
from oracle import sdlm_layer_oracle as lo
import sdlm_synth as syn

pytestmark = pytest.mark.gpu


def _ctx(lens=(5, 70, 300), D=4):
    wl = syn.Workload("layer", syn.SHAPE_TINY, len(lens), D, 0, 0, (0.9,), seed=77)
    return DeviceProblem(wl, lengths=np.asarray(lens, dtype=np.int32))


def _bf16(rng, shape, std=1.0):
    bits = syn.f32_to_bf16_bits((rng.normal(size=shape) * std).astype(np.float32))
    return bits, syn.bf16_bits_to_f32(bits).astype(np.float64), pk.bf16_tensor_from_bits(bits)


def _f64(t):
    return syn.bf16_bits_to_f32(pk.bits_from_bf16_tensor(t)).astype(np.float64)


def _check_bf16(got, ref, what, rel=2.0 ** -8):
    """One bf16 rounding of an fp32 result: within half an ulp of bf16 (2^-9 relative) plus fp32 noise."""
    err = np.abs(got - ref)
    bound = rel * np.abs(ref) + 1e-3 * np.max(np.abs(ref)) * 2.0 ** -8 + 1e-30
    assert np.all(np.isfinite(got)) and np.all(err <= bound), f"{what}: max err {err.max()} (ref max {np.abs(ref).max()})"


@pytest.mark.parametrize("rows,K,N", [(1, 64, 16), (5, 72, 48), (128, 256, 1024), (129, 128, 256), (256, 2048, 512),
                                      (33, 1000, 2512), (128, 2048, 22016), (128, 6912, 5120), (70, 2048, 8192),
                                      (128, 27648, 5120), (128, 5120, 7168)])
@pytest.mark.parametrize("extras", ["plain", "bias", "residual", "both"])
def test_linear_matches_the_oracle(rows, K, N, extras):
    if (N == 22016 or K == 27648 or N == 7168) and extras != "both":
        pytest.skip("the large shapes once")
    if K == 6912 and extras in ("bias", "residual"):
        pytest.skip("the long shape twice")
    dp = _ctx()
    rng = np.random.default_rng(rows + K + N)
    _, x64, x = _bf16(rng, (rows, K))
    _, w64, w = _bf16(rng, (N, K), std=K ** -0.5)
    _, b64, b = _bf16(rng, (N,))
    _, r64, r = _bf16(rng, (rows, N))
    use_b, use_r = extras in ("bias", "both"), extras in ("residual", "both")
    out = dp.sd.linear(x, w, b if use_b else None, r if use_r else None)
    torch.cuda.synchronize()
    assert dp.sd.device_status()[0] == 0
    ref = lo.linear(x64, w64, b64 if use_b else None, r64 if use_r else None)
    _check_bf16(_f64(out), ref, "linear")


@pytest.mark.parametrize("rows,K,n", [(128, 2048, (2048, 256, 256)), (37, 256, (64, 16, 32)), (200, 512, (256, 128, 128))])
def test_linear_with_three_outputs_matches_three_products(rows, K, n):
    """The q / k / v projections from one product over the stacked weight."""
    dp = _ctx()
    rng = np.random.default_rng(rows + K)
    _, x64, x = _bf16(rng, (rows, K))
    _, w64, w = _bf16(rng, (sum(n), K), std=K ** -0.5)
    _, b64, b = _bf16(rng, (sum(n),))
    outs = [torch.full((rows, m), 7.0, dtype=torch.bfloat16, device="cuda") for m in n]
    dp.sd.linear3(x, w, b, *outs)
    torch.cuda.synchronize()
    assert dp.sd.device_status()[0] == 0
    ref = lo.linear(x64, w64, b64)
    c = 0
    for o, m in zip(outs, n):
        _check_bf16(_f64(o), ref[:, c:c + m], "linear3")
        c += m


@pytest.mark.parametrize("rows,K,I", [(128, 2048, 11008), (9, 256, 40), (200, 512, 1024)])
def test_gated_product_matches_product_then_swiglu(rows, K, I):
    """sdlm_linear_swiglu over interleaved gate / up rows against the oracle's swiglu(linear(x, [gate ; up]))."""
    dp = _ctx()
    rng = np.random.default_rng(rows + K + I)
    _, x64, x = _bf16(rng, (rows, K))
    wb, w64, _ = _bf16(rng, (2 * I, K), std=K ** -0.5)                      # [gate rows ; up rows]
    il = np.ascontiguousarray(np.stack([wb[:I], wb[I:]], axis=1).reshape(2 * I, K))
    out = dp.sd.linear_swiglu(x, pk.bf16_tensor_from_bits(il))
    torch.cuda.synchronize()
    assert dp.sd.device_status()[0] == 0
    ref = lo.swiglu(lo.linear(x64, w64))
    _check_bf16(_f64(out), ref, "linear_swiglu", rel=2.0 ** -7)


def test_linear_in_place_on_the_residual_stream():
    dp = _ctx()
    rng = np.random.default_rng(9)
    _, x64, x = _bf16(rng, (40, 128))
    _, w64, w = _bf16(rng, (256, 128), std=0.1)
    _, r64, r = _bf16(rng, (40, 256))
    dp.sd.linear(x, w, None, r, out=r)
    torch.cuda.synchronize()
    _check_bf16(_f64(r), lo.linear(x64, w64, None, r64), "linear in place")


@pytest.mark.parametrize("rows,K,N", [(128, 2048, 2048), (128, 11008, 2048), (37, 2048, 2048), (200, 4096, 4096),
                                      (128, 2048, 4112), (9, 72, 48), (128, 256, 1024), (128, 5120, 5120),
                                      (150, 6912, 5120), (128, 2048, 6144), (64, 2048, 7168), (128, 1024, 8192),
                                      (16, 1024, 8208)])
@pytest.mark.parametrize("extras", ["plain", "both", "in place"])
def test_product_with_the_norm_of_its_rows_equals_the_two_calls(rows, K, N, extras):
    """sdlm_linear_rmsnorm against sdlm_linear followed by sdlm_rmsnorm, bit for bit (products that are cut
    along K, where the sum of the ranges and the norm share a kernel, and products that are not), and
    against the oracle's two functions."""
    dp = _ctx()
    rng = np.random.default_rng(rows + K + N + 1)
    _, x64, x = _bf16(rng, (rows, K))
    _, w64, w = _bf16(rng, (N, K), std=K ** -0.5)
    _, b64, b = _bf16(rng, (N,))
    _, r64, r = _bf16(rng, (rows, N))
    _, g64, g = _bf16(rng, (N,))
    eps = 1e-6
    use = extras != "plain"
    ref_out = dp.sd.linear(x, w, b if use else None, r if use else None)
    ref_norm = dp.sd.rmsnorm(ref_out, g, eps)
    if extras == "in place":
        res = r.clone()
        out, norm = dp.sd.linear_rmsnorm(x, w, g, eps, b, res, out=res)
    else:
        out, norm = dp.sd.linear_rmsnorm(x, w, g, eps, b if use else None, r if use else None)
    torch.cuda.synchronize()
    assert dp.sd.device_status()[0] == 0
    assert torch.equal(out, ref_out) and torch.equal(norm, ref_norm)
    o64 = lo.linear(x64, w64, b64 if use else None, r64 if use else None)
    _check_bf16(_f64(out), o64, "linear")
    _check_bf16(_f64(norm), lo.rms_norm(_f64(out), g64, eps), "norm of the stored rows")


@pytest.mark.parametrize("rows,H", [(1, 8), (7, 256), (128, 2048), (130, 5120), (3, 1000)])
def test_rmsnorm_matches_the_oracle(rows, H):
    dp = _ctx()
    rng = np.random.default_rng(rows + H)
    _, x64, x = _bf16(rng, (rows, H), std=3.0)
    _, g64, g = _bf16(rng, (H,))
    out = dp.sd.rmsnorm(x, g, 1e-6)
    torch.cuda.synchronize()
    _check_bf16(_f64(out), lo.rms_norm(x64, g64, 1e-6), "rmsnorm")


@pytest.mark.parametrize("n_heads,theta", [(4, 1.0e6), (2, 10000.0)])
def test_rope_of_the_block_uses_the_positions_after_the_cached_history(n_heads, theta):
    lens = (0, 5, 70, 300, 4000)
    dp = _ctx(lens, D=4)
    d = dp.wl.shape.head_dim
    rng = np.random.default_rng(n_heads)
    _, x64, x = _bf16(rng, (len(lens), 4, n_heads, d))
    dp.sd.rope_block(x, theta)
    torch.cuda.synchronize()
    pos = np.asarray(lens)[:, None] + np.arange(4)[None, :]
    ref = lo.rope(x64, pos, theta)
    got = _f64(x)
    # the angle is formed in fp32 on the GPU: pos * inv_freq carries a relative error of ~2^-23 * pos
    assert np.max(np.abs(got - ref)) <= 2.0 ** -8 * np.max(np.abs(ref)) + 4e-3
    # query and key rows in one launch: the same values as one launch each
    _, a64, a = _bf16(rng, (len(lens), 4, n_heads, d))
    _, b64, b = _bf16(rng, (len(lens), 4, 1, d))
    a1, b1 = a.clone(), b.clone()
    dp.sd.rope_block2(a, b, theta)
    dp.sd.rope_block(a1, theta); dp.sd.rope_block(b1, theta)
    torch.cuda.synchronize()
    assert torch.equal(a, a1) and torch.equal(b, b1)
    # with seq_ids the named slots' lengths are used
    _, y64, y = _bf16(rng, (2, 4, n_heads, d))
    ids = torch.tensor([3, 1], dtype=torch.int32).cuda()
    dp.sd.rope_block(y, theta, seq_ids=ids)
    torch.cuda.synchronize()
    ref2 = lo.rope(y64, np.array([300, 5])[:, None] + np.arange(4)[None, :], theta)
    assert np.max(np.abs(_f64(y) - ref2)) <= 2.0 ** -8 * np.max(np.abs(ref2)) + 4e-3


@pytest.mark.parametrize("batch,D,K,heads", [(3, 4, 256, (4, 1)), (40, 4, 2048, (4, 2)), (32, 4, 2048, (4, 2)), (5, 3, 2048, (16, 2)), (33, 8, 1024, (2, 2)),
                                             (32, 4, 2048, (80, 16))])
def test_qkv_product_with_rotary_equals_the_two_calls_and_the_oracle(batch, D, K, heads):
    """One call for a layer's q / k / v rows: the same bits as the product followed by the rotary call, whether
    the product is cut along K (the rotation rides on the sum of the K ranges) or not, over several row blocks,
    with and without seq_ids."""
    lens = tuple(int(v) for v in np.random.default_rng(batch).integers(0, 500, size=batch))
    dp = _ctx(lens, D=D)
    d, theta = dp.wl.shape.head_dim, 1.0e6
    hq, hk = heads
    rng = np.random.default_rng(batch + K)
    _, x64, x = _bf16(rng, (batch * D, K))
    _, w64, w = _bf16(rng, ((hq + 2 * hk) * d, K), std=K ** -0.5)
    _, b64, b = _bf16(rng, ((hq + 2 * hk) * d,))
    new = lambda h: torch.full((batch, D, h, d), 7.0, dtype=torch.bfloat16, device="cuda")
    for ids in (None, torch.tensor(np.random.default_rng(1).permutation(batch).astype(np.int32)).cuda()):
        q, k, v = new(hq), new(hk), new(hk)
        q1, k1, v1 = new(hq), new(hk), new(hk)
        dp.sd.linear3_rope(x, w, b, q, k, v, theta, seq_ids=ids)
        dp.sd.linear3(x, w, b, q1, k1, v1)
        dp.sd.rope_block2(q1, k1, theta, seq_ids=ids)
        torch.cuda.synchronize()
        assert dp.sd.device_status()[0] == 0
        assert torch.equal(q, q1) and torch.equal(k, k1) and torch.equal(v, v1)
    # against the oracle: product rounded to bf16, then the rotation (slots in the last order used)
    prod = lo.linear(x64, w64, b64)
    rb = lambda a: syn.bf16_bits_to_f32(syn.f32_to_bf16_bits(a.astype(np.float32))).astype(np.float64)
    order = ids.cpu().numpy()
    pos = np.asarray(lens)[order][:, None] + np.arange(D)[None, :]
    ref_q = lo.rope(rb(prod[:, :hq * d]).reshape(batch, D, hq, d), pos, theta)
    ref_k = lo.rope(rb(prod[:, hq * d:(hq + hk) * d]).reshape(batch, D, hk, d), pos, theta)
    for got, ref in ((q, ref_q), (k, ref_k)):
        assert np.max(np.abs(_f64(got) - ref)) <= 2.0 ** -7 * np.max(np.abs(ref)) + 4e-3
    _check_bf16(_f64(v).reshape(batch * D, -1), prod[:, (hq + hk) * d:], "v of linear3_rope")
    assert dp.sd.linear3_rope.__doc__


@pytest.mark.parametrize("rows,I", [(1, 8), (9, 1000), (128, 11008)])
def test_swiglu_matches_the_oracle(rows, I):
    dp = _ctx()
    rng = np.random.default_rng(rows + I)
    _, gu64, gu = _bf16(rng, (rows, 2 * I), std=2.0)
    out = dp.sd.swiglu(gu)
    torch.cuda.synchronize()
    _check_bf16(_f64(out), lo.swiglu(gu64), "swiglu", rel=2.0 ** -7)


def test_layer_pieces_reject_bad_arguments():
    dp = _ctx()
    x = torch.zeros((4, 60), dtype=torch.bfloat16, device="cuda")         # K not a multiple of 8
    w = torch.zeros((16, 60), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(pk.SdlmError) as e:
        dp.sd.linear(x, w)
    assert e.value.code == 3                                              # SDLM_ERR_UNSUPPORTED
    with pytest.raises(pk.SdlmError):
        dp.sd.linear(torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda"),
                     torch.zeros((8, 64), dtype=torch.bfloat16, device="cuda"))   # N < 16
    # the q / k / v product with rotary: more block rows than the context's batch, a base that is no base; nothing runs
    d = dp.wl.shape.head_dim
    n0 = dp.sd.launch_count()
    z = lambda *shape: torch.zeros(shape, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(pk.SdlmError) as e:
        dp.sd.linear3_rope(z(16, 64), z(4 * d, 64), None, z(4, 4, 2, d), z(4, 4, 1, d), z(4, 4, 1, d), 1.0e6)
    assert e.value.code == 2                                              # SDLM_ERR_SHAPE: the context holds three sequences
    with pytest.raises(pk.SdlmError) as e:
        dp.sd.linear3_rope(z(12, 64), z(4 * d, 64), None, z(3, 4, 2, d), z(3, 4, 1, d), z(3, 4, 1, d), 1.0)
    assert e.value.code == 1                                              # SDLM_ERR_INVALID_ARG
    assert dp.sd.launch_count() == n0


def test_two_layer_stack_step_matches_the_oracle_composition():
    """A tiny whole-model step: the residual stream after two layers against the oracle's float64
    composition (tolerance from the number of bf16 tensors on the way), then LM head and acceptance on the
    GPU's own final hidden state (so that the integer results are compared without accumulated drift),
    and every layer's cache grown by the same accepted rows."""
    from paper_2509_24007_b200.harness import DecoderStack, LayerWeights
    from oracle import sdlm_oracle as orc
    from oracle_side import oracle_cache, check_tokens, check_confidences, check_gamma
    shape = syn.SHAPE_TINY                                   # Hq 4, Hkv 2, d 64, H 256, V 1024
    B, D, L, I = 3, 4, 2, 512
    lens = np.array([0, 70, 200], dtype=np.int32)
    wl = syn.Workload("stack", shape, B, D, 0, 0, (0.9,), steps=4, seed=4242)
    rng = np.random.default_rng(1)
    H, Hq, Hkv, d = shape.hidden, shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    host_layers, dev_layers = [], []
    for l in range(L):
        spec = {"ln1": ((H,), 1.0, 1.0), "wq": ((Hq * d, H), 0.0, H ** -0.5), "bq": ((Hq * d,), 0.0, 0.1),
                "wk": ((Hkv * d, H), 0.0, H ** -0.5), "bk": ((Hkv * d,), 0.0, 0.1), "wv": ((Hkv * d, H), 0.0, H ** -0.5),
                "bv": ((Hkv * d,), 0.0, 0.1), "wo": ((H, Hq * d), 0.0, (Hq * d) ** -0.5), "ln2": ((H,), 1.0, 0.1),
                "wgu": ((2 * I, H), 0.0, H ** -0.5), "wdown": ((H, I), 0.0, I ** -0.5)}
        hw, dw = {}, {}
        for name, (shp, mean, std) in spec.items():
            bits = syn.f32_to_bf16_bits((mean + std * rng.normal(size=shp)).astype(np.float32))
            hw[name] = syn.bf16_bits_to_f32(bits).astype(np.float64)
            dw[name] = pk.bf16_tensor_from_bits(bits)
        host_layers.append(hw)
        dev_layers.append(LayerWeights(**dw))
    lnf_bits = syn.f32_to_bf16_bits((1.0 + 0.1 * rng.normal(size=H)).astype(np.float32))
    w_bits = syn.lm_head_weight(wl)
    prefixes = [[syn.prefix_kv(wl.with_(seed=wl.seed + 17 * l), b, int(lens[b])) for b in range(B)] for l in range(L)]
    stack = DecoderStack(wl, L, I, lens, dev_layers, pk.bf16_tensor_from_bits(lnf_bits), pk.bf16_tensor_from_bits(w_bits),
                         lambda l, b, n: tuple(pk.bf16_tensor_from_bits(t) for t in prefixes[l][b]))
    caches = [oracle_cache(wl, lens, stack.num_pages, stack.mpps, prefixes[l]) for l in range(L)]
    out = StepOutputs_like(stack)
    for step in range(2):
        h0_bits = syn.f32_to_bf16_bits(rng.normal(size=(B, D, H)).astype(np.float32))
        stack.step(pk.bf16_tensor_from_bits(h0_bits), wl.tau, out)
        torch.cuda.synchronize()
        assert all(sd.device_status()[0] == 0 for sd in stack.ctx)
        h_ref, k_ref, v_ref = lo.decoder_stack_hidden(syn.bf16_bits_to_f32(h0_bits).astype(np.float64), host_layers, caches,
                                                     range(B), Hq, Hkv, d, stack.EPS, stack.THETA)
        # The oracle is float64 throughout; the library keeps a bf16 tensor between two calls.  Along the
        # longest chain of a layer there are 8 such roundings (norm, q/k/v, rotary, attention output,
        # stream after the output projection, norm, gated activation, stream after the down projection),
        # each at most 2^-9 of the largest magnitude and adding up linearly at worst; one more unit stands
        # for fp32 accumulation order and the approximate exponentials.
        unit = 2.0 ** -9
        h_gpu = _f64(stack.h)
        scale = np.max(np.abs(h_ref))
        assert np.max(np.abs(h_gpu - h_ref)) <= (8 * L + 1) * unit * scale, (np.max(np.abs(h_gpu - h_ref)), scale)
        for l in range(L):                                   # the rows each layer is about to commit
            for got, ref, n_round in ((stack.k[l], k_ref[l], 8 * l + 3), (stack.v[l], v_ref[l], 8 * l + 2)):
                err = np.max(np.abs(_f64(got) - ref))
                assert err <= (n_round + 1) * unit * np.max(np.abs(ref)), (l, err, np.max(np.abs(ref)))
        # head and acceptance: from the GPU's own final normalised hidden state
        x_bits = pk.bits_from_bf16_tensor(stack.x).reshape(B, D, H)
        stats = orc.lm_head_statistics(x_bits, w_bits)
        flagged = []
        check_tokens(out.token.cpu().numpy(), stats, flagged)
        check_confidences(out.p_top1.cpu().numpy(), out.entropy.cpu().numpy(), stats)
        conf = stats.p_top1.reshape(B, D)
        for l in range(L):
            kb, vb = pk.bits_from_bf16_tensor(stack.k[l]), pk.bits_from_bf16_tensor(stack.v[l])
            res = orc.accept_and_commit(caches[l], range(B), stats.token.reshape(B, D), conf, wl.tau, kb, vb)
            t = stack.ctx[l].kv_tables()
            assert np.array_equal(t["page_table"], caches[l].page_table) and np.array_equal(t["seq_len"], caches[l].seq_len)
            for b in range(B):
                k, v = stack.ctx[l].kv_gather(b, int(caches[l].seq_len[b]))
                ok, ov = caches[l].gather_fast(b)
                assert np.array_equal(pk.bits_from_bf16_tensor(k), ok) and np.array_equal(pk.bits_from_bf16_tensor(v), ov)
        assert check_gamma(out.accepted_len.cpu().numpy(), res, flagged) == 0


def StepOutputs_like(stack):
    from paper_2509_24007_b200.harness import StepOutputs
    wl, s, dev = stack.wl, stack.wl.shape, stack.ctx[0].device
    B, D = wl.batch, wl.block
    return StepOutputs(torch.empty((B, D, s.n_q_heads, s.head_dim), dtype=torch.bfloat16, device=dev),
                       torch.empty((B, D), dtype=torch.int32, device=dev), torch.empty((B, D), dtype=torch.float32, device=dev),
                       torch.empty((B, D), dtype=torch.float32, device=dev), torch.empty(B, dtype=torch.int32, device=dev),
                       torch.empty((B, D), dtype=torch.int32, device=dev))
