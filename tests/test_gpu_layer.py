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
                                      (33, 1000, 2512), (128, 2048, 22016)])
@pytest.mark.parametrize("extras", ["plain", "bias", "residual", "both"])
def test_linear_matches_the_oracle(rows, K, N, extras):
    if N == 22016 and extras != "both":
        pytest.skip("the large shape once")
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


def test_linear_in_place_on_the_residual_stream():
    dp = _ctx()
    rng = np.random.default_rng(9)
    _, x64, x = _bf16(rng, (40, 128))
    _, w64, w = _bf16(rng, (256, 128), std=0.1)
    _, r64, r = _bf16(rng, (40, 256))
    dp.sd.linear(x, w, None, r, out=r)
    torch.cuda.synchronize()
    _check_bf16(_f64(r), lo.linear(x64, w64, None, r64), "linear in place")


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
    # with seq_ids the named slots' lengths are used
    _, y64, y = _bf16(rng, (2, 4, n_heads, d))
    ids = torch.tensor([3, 1], dtype=torch.int32).cuda()
    dp.sd.rope_block(y, theta, seq_ids=ids)
    torch.cuda.synchronize()
    ref2 = lo.rope(y64, np.array([300, 5])[:, None] + np.arange(4)[None, :], theta)
    assert np.max(np.abs(_f64(y) - ref2)) <= 2.0 ** -8 * np.max(np.abs(ref2)) + 4e-3


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
