"""GPU parity: split-KV paged block-decode attention against the oracle's dense fp64 softmax."""
import numpy as np
import pytest
import torch

import paper_2509_24007_b200 as pk
from paper_2509_24007_b200.harness import DeviceProblem
from oracle import sdlm_oracle as orc
import sdlm_synth as syn
from oracle_side import check_attention

pytestmark = pytest.mark.gpu


def _attn_case(shape, lens, D, seed, scale_note=None):
    lens = np.asarray(lens, dtype=np.int32)
    wl = syn.Workload("attn", shape, len(lens), D, 0, 0, (0.9,), seed=seed)
    dp = DeviceProblem(wl, w_bits=np.zeros((shape.vocab, shape.hidden), np.uint16), lengths=lens)
    x = dp.block(0)
    out = dp.sd.block_attn(x.q, x.k_blk, x.v_blk)
    torch.cuda.synchronize()
    assert dp.sd.device_status()[0] == 0
    pk_, pv_ = zip(*dp.prefix)
    ref = orc.block_attention(x.host.q, x.host.k_blk, x.host.v_blk, pk_, pv_)
    return check_attention(pk.bits_from_bf16_tensor(out), ref), dp, x, out


@pytest.mark.parametrize("Hq,Hkv,d", [(4, 2, 64), (2, 2, 128), (16, 2, 128), (10, 2, 128), (8, 1, 64)])
@pytest.mark.parametrize("D", [1, 2, 4, 8])
def test_attention_ragged_prefixes(Hq, Hkv, d, D):
    shape = syn.Shape(Hq, Hkv, d, 64, 64)
    lens = [0, 1, 63, 64, 65, 127, 128, 300, 1000]
    _attn_case(shape, lens, D, seed=200 + Hq + D)


def test_attention_long_prefix_is_split_across_many_items():
    shape = syn.Shape(16, 2, 128, 64, 64)
    err, dp, x, out = _attn_case(shape, [20000, 3], 8, seed=31)
    # same inputs, second launch: bit-identical (fixed merge order)
    out2 = dp.sd.block_attn(x.q, x.k_blk, x.v_blk)
    assert torch.equal(out, out2)


def test_attention_with_seq_ids_reads_the_named_slots():
    shape = syn.SHAPE_TINY
    lens = np.array([70, 5, 190], dtype=np.int32)
    wl = syn.Workload("attn_ids", shape, 3, 4, 0, 0, (0.9,), seed=33)
    dp = DeviceProblem(wl, w_bits=np.zeros((shape.vocab, shape.hidden), np.uint16), lengths=lens)
    ids = np.array([2, 0], dtype=np.int32)
    x = syn.block_inputs(wl.with_(batch=2), dp.w_bits)
    out = dp.sd.block_attn(pk.bf16_tensor_from_bits(x.q), pk.bf16_tensor_from_bits(x.k_blk),
                           pk.bf16_tensor_from_bits(x.v_blk), seq_ids=torch.from_numpy(ids).cuda())
    ref = orc.block_attention(x.q, x.k_blk, x.v_blk, [dp.prefix[2][0], dp.prefix[0][0]],
                              [dp.prefix[2][1], dp.prefix[0][1]])
    check_attention(pk.bits_from_bf16_tensor(out), ref)


def test_attention_ignores_garbage_beyond_the_sequence_end():
    """Rows of the last page past seq_len hold arbitrary bits (here NaN patterns): they must not leak."""
    shape = syn.SHAPE_TINY
    lens = np.array([70], dtype=np.int32)
    wl = syn.Workload("attn_nan", shape, 1, 4, 0, 0, (0.9,), seed=34)
    dp = DeviceProblem(wl, w_bits=np.zeros((shape.vocab, shape.hidden), np.uint16), lengths=lens)
    dp.sd._pool.fill_(0xFF)                      # every bf16 in the pool becomes a NaN pattern
    dp.sd.kv_reset(dp.free_list)
    k, v = dp.prefix[0]
    dp.sd.kv_add_seq(0, pk.bf16_tensor_from_bits(k), pk.bf16_tensor_from_bits(v))
    x = dp.block(0)
    out = dp.sd.block_attn(x.q, x.k_blk, x.v_blk)
    ref = orc.block_attention(x.host.q, x.host.k_blk, x.host.v_blk, [k], [v])
    check_attention(pk.bits_from_bf16_tensor(out), ref)


@pytest.mark.parametrize("D", [4, 8])
def test_attention_with_scores_that_keep_outgrowing_the_row_reference(D):
    """Scores rise steadily along the sequence (by far more than 2^32 per 128 keys), and fall again
    for a second sequence: the kernel has to move its softmax references many times, or never."""
    shape = syn.Shape(16, 2, 128, 64, 64)
    lens = np.array([700, 333], dtype=np.int32)
    wl = syn.Workload("attn_rebase", shape, 2, D, 0, 0, (0.9,), seed=36)
    dp = DeviceProblem(wl, w_bits=np.zeros((shape.vocab, shape.hidden), np.uint16), lengths=lens)
    x = syn.block_inputs(wl, dp.w_bits)
    q = syn.bf16_bits_to_f32(x.q) * 0.05
    q[..., 0] = 8.0                                           # every query looks along coordinate 0
    prefix = []
    for b, n in enumerate(lens):
        k, v = dp.prefix[b]
        kf = syn.bf16_bits_to_f32(k) * 0.05
        ramp = np.arange(n, dtype=np.float32) * 0.5
        kf[:, :, 0] = (ramp if b == 0 else ramp[::-1])[:, None]
        prefix.append((syn.f32_to_bf16_bits(kf), v))
    dp.prefix = prefix
    dp.reset_cache()
    q_bits = syn.f32_to_bf16_bits(q)
    out = dp.sd.block_attn(pk.bf16_tensor_from_bits(q_bits), pk.bf16_tensor_from_bits(x.k_blk),
                           pk.bf16_tensor_from_bits(x.v_blk))
    torch.cuda.synchronize()
    assert dp.sd.device_status()[0] == 0
    ref = orc.block_attention(q_bits, x.k_blk, x.v_blk, [a for a, _ in prefix], [b for _, b in prefix])
    check_attention(pk.bits_from_bf16_tensor(out), ref)


@pytest.mark.parametrize("cost", [0, 3, 17, 64])
def test_attention_schedule_item_cost_does_not_change_results(cost):
    from paper_2509_24007_b200.binding import OPT_ATTN_ITEM_COST
    shape = syn.Shape(16, 2, 128, 64, 64)
    lens = np.array([0, 1, 64, 700, 129, 2500, 63, 300, 5], dtype=np.int32)
    wl = syn.Workload("attn_cost", shape, len(lens), 4, 0, 0, (0.9,), seed=37)
    dp = DeviceProblem(wl, w_bits=np.zeros((shape.vocab, shape.hidden), np.uint16), lengths=lens)
    dp.sd.set_option(OPT_ATTN_ITEM_COST, cost)
    x = dp.block(0)
    out = dp.sd.block_attn(x.q, x.k_blk, x.v_blk)
    torch.cuda.synchronize()
    assert dp.sd.device_status()[0] == 0
    pk_, pv_ = zip(*dp.prefix)
    check_attention(pk.bits_from_bf16_tensor(out), orc.block_attention(x.host.q, x.host.k_blk, x.host.v_blk, pk_, pv_))


def test_attention_many_short_sequences_many_items_per_thread_block():
    """600 sequences, most of them shorter than a page: more (sequence, head) pairs than thread blocks,
    several items per thread block, a long prefix-sum table in shared memory."""
    shape = syn.Shape(4, 2, 64, 64, 64)
    rng = np.random.default_rng(7)
    lens = rng.integers(0, 200, size=600).astype(np.int32)
    lens[::37] = 0
    _attn_case(shape, lens, 2, seed=38)


def test_attention_rejects_bad_arguments():
    shape = syn.SHAPE_TINY
    wl = syn.Workload("attn_bad", shape, 2, 4, 8, 8, (0.9,), seed=35)
    dp = DeviceProblem(wl, w_bits=np.zeros((shape.vocab, shape.hidden), np.uint16))
    x = dp.block(0)
    big = torch.zeros((3, 4, 4, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(pk.SdlmError) as e:
        dp.sd.block_attn(big, x.k_blk, x.v_blk)
    assert e.value.code == 2
