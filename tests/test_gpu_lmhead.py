"""GPU parity: fused LM head -> softmax statistics against the oracle's two-pass fp64 rows."""
import numpy as np
import pytest
import torch

import paper_2509_24007_b200 as pk
from paper_2509_24007_b200.binding import OPT_LMHEAD_KERNEL
from oracle import sdlm_oracle as orc
import sdlm_synth as syn
from oracle_side import check_confidences, check_tokens

pytestmark = pytest.mark.gpu

KERNELS = {"mma": 1, "umma": 2}


def _ctx(shape, rows):
    cfg = pk.SdlmConfig(shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.hidden, shape.vocab,
                        num_pages=4, max_batch=(rows + 7) // 8, max_pages_per_seq=2, max_block=8)
    return pk.Sdlm(cfg)


def _run(sd, hidden_bits, w_bits, kernel):
    sd.set_option(OPT_LMHEAD_KERNEL, KERNELS[kernel])
    rows = hidden_bits.shape[0]
    mx = torch.empty(rows, device="cuda"); lse = torch.empty(rows, device="cuda")
    tok, p, ent = sd.lmhead_confidence(pk.bf16_tensor_from_bits(hidden_bits), pk.bf16_tensor_from_bits(w_bits),
                                       max_logit=mx, lse=lse)
    torch.cuda.synchronize()
    assert sd.device_status()[0] == 0
    return tok.cpu().numpy(), p.cpu().numpy(), ent.cpu().numpy(), mx.cpu().numpy(), lse.cpu().numpy()


def _compare(out, stats):
    tok, p, ent, mx, lse = out
    report = []
    check_tokens(tok, stats, report)
    check_confidences(p, ent, stats)
    assert np.max(np.abs(mx - stats.max_logit)) < 2e-3
    assert np.max(np.abs(lse - stats.lse)) < 2e-3
    return report


@pytest.mark.parametrize("kernel", ["mma", "umma"])
@pytest.mark.parametrize("rows,H,V", [(4, 256, 1024), (1, 64, 16), (7, 72, 1000), (128, 320, 2500), (129, 256, 4099),
                                      (256, 128, 3001), (33, 2048, 5000), (200, 1000, 777)])
def test_lmhead_random_shapes(kernel, rows, H, V):
    shape = syn.Shape(4, 2, 64, H, V)
    wl = syn.Workload("lm", shape, rows, 1, 0, 0, (0.9,), seed=100 + rows)
    w_bits = syn.lm_head_weight(wl)
    x = syn.block_inputs(wl, w_bits)
    hidden = x.hidden.reshape(rows, H)
    stats = orc.lm_head_statistics(hidden, w_bits)
    sd = _ctx(shape, rows)
    _compare(_run(sd, hidden, w_bits, kernel), stats)
    # confident positions recover the planted token
    conf = stats.p_top1 > 0.9
    assert np.array_equal(stats.token[conf], x.target.reshape(-1)[conf])


@pytest.mark.parametrize("kernel", ["mma", "umma"])
def test_lmhead_ties_and_degenerate_rows(kernel):
    """Exact ties resolve to the lowest index; a zero hidden state gives the uniform distribution."""
    H, V, rows = 64, 4000, 5
    shape = syn.Shape(4, 2, 64, H, V)
    rng = np.random.default_rng(5)
    w = rng.integers(-3, 4, size=(V, H)).astype(np.float32)            # small integers: exact in bf16 and fp32
    w[3000] = w[17]; w[3999] = w[17]                                    # three identical rows -> exact ties
    hid = np.zeros((rows, H), np.float32)
    hid[1] = w[17] * 2                                                  # row 17 (and its copies) wins
    hid[2] = rng.integers(-2, 3, size=H)
    hid[3] = w[3999] * 0.5
    hid[4] = -w[1234]
    w_bits, h_bits = syn.f32_to_bf16_bits(w), syn.f32_to_bf16_bits(hid)
    stats = orc.lm_head_statistics(h_bits, w_bits)
    out = _run(_ctx(shape, rows), h_bits, w_bits, kernel)
    assert out[0][0] == 0 and abs(out[1][0] - 1.0 / V) < 1e-7 and abs(out[2][0] - np.log(V)) < 1e-4
    assert out[0][1] == 17 and out[0][3] == 17
    assert np.array_equal(out[0], stats.token)                          # integer logits: no rounding, exact ties
    check_confidences(out[1], out[2], stats)


def test_lmhead_cfg0_and_kernels_agree():
    wl = syn.CONFIGS["cfg0"].with_(batch=16)
    w_bits = syn.lm_head_weight(wl)
    x = syn.block_inputs(wl, w_bits)
    hidden = x.hidden.reshape(-1, wl.shape.hidden)
    stats = orc.lm_head_statistics(hidden, w_bits)
    sd = _ctx(wl.shape, hidden.shape[0])
    a = _run(sd, hidden, w_bits, "mma")
    b = _run(sd, hidden, w_bits, "umma")
    _compare(a, stats); _compare(b, stats)
    assert np.array_equal(a[0], b[0])
    # run-to-run determinism: the merge order is fixed
    c = _run(sd, hidden, w_bits, "umma")
    assert all(np.array_equal(u, v) for u, v in zip(b, c))


def test_lmhead_rejects_bad_arguments():
    shape = syn.SHAPE_TINY
    sd = _ctx(shape, 8)
    h = torch.zeros((8, shape.hidden), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((shape.vocab, shape.hidden), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(pk.SdlmError) as e:
        sd.lmhead_confidence(torch.zeros((9, shape.hidden), dtype=torch.bfloat16, device="cuda"), w)
    assert e.value.code == 2
    with pytest.raises(TypeError):
        sd.lmhead_confidence(h.float(), w)
    sd.lmhead_confidence(h, w)
