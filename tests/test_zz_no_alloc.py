"""GPU check of sdlm_lmhead_confidence_static, the LM-head entry point for callers that must not
allocate device memory (their pool is sealed, or their policy forbids allocation inside the step).

It keeps its scratch in a fixed array inside the library, so every call on a device shares that
array and sees what the previous call left there.  The test therefore makes two calls in a row, of
different sizes and with different inputs, and compares each with sdlm_lmhead_confidence (which
uses the context's workspace) on the same inputs, and with the CPU oracle's two-pass statistics.
This file sorts last on purpose: a run that stops at the first failure has then already run every
other test.
"""
import numpy as np
import pytest
import torch

import paper_2509_24007_b200 as pk
import sdlm_synth as syn
from oracle import sdlm_oracle as orc
from oracle_side import TOL_CONF, TOL_ENTROPY, check_confidences, check_tokens

pytestmark = pytest.mark.gpu


def _inputs(rows, H, V, seed):
    shape = syn.Shape(4, 2, 64, H, V)
    wl = syn.Workload("static", shape, rows, 1, 0, 0, (0.9,), seed=seed)
    w_bits = syn.lm_head_weight(wl)
    hidden = syn.block_inputs(wl, w_bits).hidden.reshape(rows, H)
    return (hidden, w_bits), pk.bf16_tensor_from_bits(hidden), pk.bf16_tensor_from_bits(w_bits)


def _outputs(rows):
    dev = "cuda"
    return (torch.full((rows,), -7, dtype=torch.int32, device=dev), torch.full((rows,), -1.0, device=dev),
            torch.full((rows,), -1.0, device=dev), torch.full((rows,), -1.0, device=dev),
            torch.full((rows,), -1.0, device=dev))


def test_static_scratch_entry_matches_workspace_entry_on_two_calls_in_a_row():
    H, V = 512, 20011
    shape = syn.Shape(4, 2, 64, H, V)
    sd = pk.Sdlm(pk.SdlmConfig(shape.n_q_heads, shape.n_kv_heads, shape.head_dim, H, V, num_pages=4, max_batch=32,
                               max_pages_per_seq=2, max_block=8))
    for rows, seed in ((200, 901), (7, 902)):        # the second, smaller call runs over the first call's leftovers
        (hidden_bits, w_bits), hidden, w = _inputs(rows, H, V, seed)
        ref = _outputs(rows)
        sd.lmhead_confidence(hidden, w, ref[0], ref[1], ref[2], max_logit=ref[3], lse=ref[4])
        got = _outputs(rows)
        sd.lmhead_confidence_static(hidden, w, got[0], got[1], got[2], max_logit=got[3], lse=got[4])
        torch.cuda.synchronize()
        assert sd.device_status()[0] == 0
        assert torch.equal(got[0], ref[0])
        assert float((got[1] - ref[1]).abs().max()) <= TOL_CONF
        assert float((got[2] - ref[2]).abs().max()) <= TOL_ENTROPY
        assert float((got[3] - ref[3]).abs().max()) <= 2e-3 and float((got[4] - ref[4]).abs().max()) <= 2e-3
        assert int(got[0].min()) >= 0 and float(got[1].min()) > 0.0
        # and against the oracle itself, on this shape
        stats = orc.lm_head_statistics(hidden_bits.reshape(rows, 1, H), w_bits)
        flagged = []
        check_tokens(got[0].cpu().numpy(), stats, flagged)
        check_confidences(got[1].cpu().numpy(), got[2].cpu().numpy(), stats)
        assert float(np.max(np.abs(got[3].cpu().numpy() - stats.max_logit))) <= 2e-3


def test_static_scratch_entry_rejects_sizes_beyond_its_array():
    shape = syn.Shape(4, 2, 64, 256, 1024)
    sd = pk.Sdlm(pk.SdlmConfig(shape.n_q_heads, shape.n_kv_heads, shape.head_dim, 256, 1024, num_pages=4, max_batch=64,
                               max_pages_per_seq=2, max_block=8))
    rows = 257                                        # the context allows 512 rows, the fixed array 256
    hidden = torch.zeros((rows, 256), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((1024, 256), dtype=torch.bfloat16, device="cuda")
    out = _outputs(rows)
    with pytest.raises(pk.SdlmError) as e:
        sd.lmhead_confidence_static(hidden, w, out[0], out[1], out[2])
    assert e.value.code == 2
    torch.cuda.synchronize()
    assert int(out[0][0]) == -7                       # nothing was enqueued
