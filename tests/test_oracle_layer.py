"""Pins for the layer oracle (linear, RMSNorm, rotary embedding, SwiGLU)."""
import numpy as np
import pytest
import torch

from oracle import sdlm_layer_oracle as lo


def test_linear_is_torch_matmul_and_identity_weights_copy_the_input():
    rng = np.random.default_rng(0)
    x, w, b, r = rng.normal(size=(5, 24)), rng.normal(size=(16, 24)), rng.normal(size=16), rng.normal(size=(5, 16))
    ref = torch.from_numpy(x) @ torch.from_numpy(w).T + torch.from_numpy(b) + torch.from_numpy(r)
    assert np.allclose(lo.linear(x, w, b, r), ref.numpy(), rtol=0, atol=1e-13)
    assert np.array_equal(lo.linear(x, np.eye(24)), x)
    assert np.allclose(lo.linear(x, w), (torch.from_numpy(x) @ torch.from_numpy(w).T).numpy(), rtol=0, atol=1e-13)


def test_rms_norm_against_torch_constant_rows_and_rescaling():
    rng = np.random.default_rng(1)
    x, g = rng.normal(size=(7, 40)), rng.normal(size=40)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x), (40,), torch.from_numpy(g), 1e-6).numpy()
    assert np.allclose(lo.rms_norm(x, g, 1e-6), ref, rtol=0, atol=1e-13)
    const = np.full((2, 16), -3.0)
    assert np.allclose(lo.rms_norm(const, np.ones(16), 0.0), -1.0)               # x / |x|
    assert np.allclose(lo.rms_norm(17.0 * x, g, 0.0), lo.rms_norm(x, g, 0.0), rtol=1e-13, atol=0)   # scale-free when eps = 0


def test_rope_is_a_complex_rotation_of_the_pairs_and_preserves_norms():
    rng = np.random.default_rng(2)
    d, theta = 16, 10000.0
    x = rng.normal(size=(3, 4, 2, d))                         # [B, D, heads, d]
    pos = rng.integers(0, 5000, size=(3, 4))
    y = lo.rope(x, pos, theta)
    z = x[..., :d // 2] + 1j * x[..., d // 2:]
    ang = pos[..., None, None] * theta ** (-2.0 * np.arange(d // 2) / d)
    zr = z * np.exp(1j * ang)
    assert np.allclose(y[..., :d // 2], zr.real, atol=1e-12) and np.allclose(y[..., d // 2:], zr.imag, atol=1e-12)
    assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-12)
    assert np.array_equal(lo.rope(x, np.zeros((3, 4)), theta), x)


def test_rope_scores_depend_on_the_position_difference_only():
    rng = np.random.default_rng(3)
    d, theta = 32, 1.0e6
    q, k = rng.normal(size=(1, 1, 1, d)), rng.normal(size=(1, 1, 1, d))
    def score(m, n):
        return float(np.sum(lo.rope(q, np.array([[m]]), theta) * lo.rope(k, np.array([[n]]), theta)))
    assert abs(score(10, 3) - score(1007, 1000)) < 1e-9
    assert abs(score(5, 5) - float(np.sum(q * k))) < 1e-12
    assert abs(score(10, 3) - score(3, 10)) > 1e-6            # not symmetric: the sign of the offset matters


def test_swiglu_against_torch_silu_and_limits():
    rng = np.random.default_rng(4)
    gu = rng.normal(size=(6, 20)) * 3
    ref = torch.nn.functional.silu(torch.from_numpy(gu[:, :10])) * torch.from_numpy(gu[:, 10:])
    assert np.allclose(lo.swiglu(gu), ref.numpy(), rtol=0, atol=1e-14)
    assert np.array_equal(lo.swiglu(np.concatenate([np.zeros((1, 4)), np.ones((1, 4))], axis=1)), np.zeros((1, 4)))
    big = np.concatenate([np.full((1, 2), 50.0), np.full((1, 2), 2.5)], axis=1)
    assert np.allclose(lo.swiglu(big), 125.0)                 # silu(g) -> g for large g
    neg = np.concatenate([np.full((1, 2), -50.0), np.full((1, 2), 2.5)], axis=1)
    assert np.all(np.abs(lo.swiglu(neg)) < 1e-18)             # and -> 0 for very negative g


def test_bf16_rounding_helper_is_nearest_even():
    vals = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 2 ** -7, 1.0 + 3 * 2 ** -8, -0.3, 3.0e38])
    want = torch.tensor(vals, dtype=torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(lo.round_bf16(vals), want)
    bits = torch.tensor(vals, dtype=torch.float32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(lo.to_bits(vals), bits)


# ---- the composition of a whole decoder layer / stack -------------------------------------------------
from oracle import sdlm_oracle as orc
import sdlm_synth as syn


def _tiny_stack(seed, B=3, D=3, Hq=4, Hkv=2, d=8, H=24, I=40, L=1, lens=(0, 5, 70)):
    rng = np.random.default_rng(seed)
    layers = []
    for _ in range(L):
        layers.append({"ln1": 1.0 + 0.2 * rng.normal(size=H), "wq": rng.normal(size=(Hq * d, H)) * H ** -0.5,
                       "bq": 0.1 * rng.normal(size=Hq * d), "wk": rng.normal(size=(Hkv * d, H)) * H ** -0.5,
                       "bk": 0.1 * rng.normal(size=Hkv * d), "wv": rng.normal(size=(Hkv * d, H)) * H ** -0.5,
                       "bv": 0.1 * rng.normal(size=Hkv * d), "wo": rng.normal(size=(H, Hq * d)) * (Hq * d) ** -0.5,
                       "ln2": 1.0 + 0.2 * rng.normal(size=H), "wgu": rng.normal(size=(2 * I, H)) * H ** -0.5,
                       "wdown": rng.normal(size=(H, I)) * I ** -0.5})
    caches = []
    for _ in range(L):
        c = orc.PagedKVCache(16, 64, Hkv, d, B, 4, np.arange(16, dtype=np.int32))
        for b, n in enumerate(lens):
            c.add_sequence_fast(b, syn.f32_to_bf16_bits(rng.normal(size=(n, Hkv, d)).astype(np.float32)),
                                syn.f32_to_bf16_bits(rng.normal(size=(n, Hkv, d)).astype(np.float32)))
        caches.append(c)
    h0 = rng.normal(size=(B, D, H))
    return h0, layers, caches, dict(n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, eps=1e-6, theta=1.0e4)


def _torch_layer(h0, w, cache, Hq, Hkv, d, eps, theta):
    """One pre-norm decoder layer written from torch's float64 routines (rms_norm, linear, silu,
    scaled_dot_product_attention with the KV heads repeated) and a complex rotary embedding."""
    F = torch.nn.functional
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float64))
    B, D, H = h0.shape
    h = t(h0)
    x = F.rms_norm(h, (H,), t(w["ln1"]), eps)
    q = F.linear(x, t(w["wq"]), t(w["bq"])).view(B, D, Hq, d)
    k = F.linear(x, t(w["wk"]), t(w["bk"])).view(B, D, Hkv, d)
    v = F.linear(x, t(w["wv"]), t(w["bv"])).view(B, D, Hkv, d)
    inv = theta ** (-2.0 * torch.arange(d // 2, dtype=torch.float64) / d)
    attn = torch.zeros(B, D, Hq, d, dtype=torch.float64)
    for b in range(B):
        P = int(cache.seq_len[b])
        ang = (P + torch.arange(D, dtype=torch.float64))[:, None, None] * inv
        rot = torch.polar(torch.ones_like(ang), ang)
        turn = lambda a: torch.cat([(torch.complex(a[..., :d // 2], a[..., d // 2:]) * rot).real,
                                    (torch.complex(a[..., :d // 2], a[..., d // 2:]) * rot).imag], dim=-1)
        qb, kb = turn(q[b]), turn(k[b])
        pk, pv = cache.gather_fast(b)
        keys = torch.cat([t(orc.widen(pk)), kb]).repeat_interleave(Hq // Hkv, dim=1)      # [P + D, Hq, d]
        vals = torch.cat([t(orc.widen(pv)), v[b]]).repeat_interleave(Hq // Hkv, dim=1)
        o = F.scaled_dot_product_attention(qb.transpose(0, 1), keys.transpose(0, 1), vals.transpose(0, 1))  # no mask
        attn[b] = o.transpose(0, 1)
    h = h + F.linear(attn.reshape(B, D, Hq * d), t(w["wo"]))
    x2 = F.rms_norm(h, (H,), t(w["ln2"]), eps)
    gu = F.linear(x2, t(w["wgu"]))
    I = gu.shape[-1] // 2
    h = h + F.linear(F.silu(gu[..., :I]) * gu[..., I:], t(w["wdown"]))
    return h.numpy().reshape(B * D, H)


def test_block_attention_values_is_the_bit_pattern_oracle_on_bf16_inputs():
    rng = np.random.default_rng(5)
    B, D, Hq, Hkv, d = 2, 3, 4, 2, 16
    bits = lambda *s: syn.f32_to_bf16_bits(rng.normal(size=s).astype(np.float32))
    q, k, v = bits(B, D, Hq, d), bits(B, D, Hkv, d), bits(B, D, Hkv, d)
    pk, pv = [bits(n, Hkv, d) for n in (0, 37)], [bits(n, Hkv, d) for n in (0, 37)]
    a = lo.block_attention_values(orc.widen(q), orc.widen(k), orc.widen(v), [orc.widen(x) for x in pk], [orc.widen(x) for x in pv])
    assert np.allclose(a, orc.block_attention(q, k, v, pk, pv), rtol=0, atol=1e-14)


def test_decoder_layer_composition_against_a_layer_written_from_torch_routines():
    h0, layers, caches, kw = _tiny_stack(11)
    h, k_rows, v_rows = lo.decoder_stack_hidden(h0, layers, caches, range(3), **kw)
    ref = _torch_layer(h0, layers[0], caches[0], kw["n_q_heads"], kw["n_kv_heads"], kw["head_dim"], kw["eps"], kw["theta"])
    assert np.max(np.abs(h - ref)) <= 1e-11 * max(1.0, np.max(np.abs(ref)))
    assert h.dtype == np.float64 and k_rows[0].shape == (3, 3, 2, 8) and v_rows[0].shape == (3, 3, 2, 8)
    # nothing is rounded on the way: moving an input by far less than a bf16 step moves the output
    h2, _, _ = lo.decoder_stack_hidden(h0 * (1.0 + 1e-9), layers, caches, range(3), **kw)
    assert 0 < np.max(np.abs(h2 - h)) < 1e-6


def test_identity_projections_and_a_zero_mlp_reduce_a_layer_to_h_plus_attention():
    Hq = Hkv = 3; d = 8; H = Hq * d
    h0, layers, caches, kw = _tiny_stack(12, Hq=Hq, Hkv=Hkv, d=d, H=H)
    w = layers[0]
    w.update(ln1=np.ones(H), wq=np.eye(H), wk=np.eye(H), wv=np.eye(H), bq=np.zeros(H), bk=np.zeros(H), bv=np.zeros(H),
             wo=np.eye(H), wdown=np.zeros_like(w["wdown"]))
    h, k_rows, v_rows = lo.decoder_stack_hidden(h0, layers, caches, range(3), **kw)
    x = lo.rms_norm(h0.reshape(9, H), np.ones(H), kw["eps"]).reshape(3, 3, Hq, d)
    pos = np.array([0, 5, 70])[:, None] + np.arange(3)[None, :]
    xr = lo.rope(x, pos, kw["theta"])
    hist = [caches[0].gather_fast(b) for b in range(3)]
    attn = lo.block_attention_values(xr, xr, x, [orc.widen(a) for a, _ in hist], [orc.widen(b) for _, b in hist])
    assert np.allclose(h, h0.reshape(9, H) + attn.reshape(9, H), rtol=0, atol=1e-13)
    assert np.allclose(k_rows[0], xr, atol=1e-14) and np.allclose(v_rows[0], x, atol=1e-14)


def test_zero_output_and_down_projections_leave_the_stream_and_two_layers_are_one_layer_twice():
    h0, layers, caches, kw = _tiny_stack(13, L=2)
    dead = [dict(w, wo=np.zeros_like(w["wo"]), wdown=np.zeros_like(w["wdown"])) for w in layers]
    h, _, _ = lo.decoder_stack_hidden(h0, dead, caches, range(3), **kw)
    assert np.array_equal(h, h0.reshape(9, -1))
    both, k2, _ = lo.decoder_stack_hidden(h0, layers, caches, range(3), **kw)
    first, _, _ = lo.decoder_stack_hidden(h0, layers[:1], caches[:1], range(3), **kw)
    second, k_second, _ = lo.decoder_stack_hidden(first.reshape(h0.shape), layers[1:], caches[1:], range(3), **kw)
    assert np.array_equal(both, second) and np.array_equal(k2[1], k_second[0])
    ref = _torch_layer(first.reshape(h0.shape), layers[1], caches[1], kw["n_q_heads"], kw["n_kv_heads"], kw["head_dim"],
                       kw["eps"], kw["theta"])
    assert np.max(np.abs(both - ref)) <= 1e-11 * max(1.0, np.max(np.abs(ref)))
