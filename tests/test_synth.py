"""The shared input generators: deterministic, correctly rounded, shaped as documented."""
import numpy as np
import torch

import sdlm_synth as syn


def test_bf16_rounding_matches_library_conversion():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.normal(size=4096).astype(np.float32) * 10,
                        np.array([1.00390625, 1.01171875, -1.00390625, 0.0, 3.0e38], np.float32)])
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(syn.f32_to_bf16_bits(x), ref)
    back = syn.bf16_bits_to_f32(ref)
    assert np.array_equal(back, torch.from_numpy(x).to(torch.bfloat16).float().numpy())


def test_draws_are_pure_functions_of_seed_and_ids():
    a = syn.normal_bf16(5, 6, (3, 1000), sub=2)
    b = syn.normal_bf16(5, 6, (3, 1000), sub=2)
    c = syn.normal_bf16(5, 6, (3, 1000), sub=3)
    assert np.array_equal(a, b) and not np.array_equal(a, c)
    big = syn.normal_bf16(1, 1, (syn._CHUNK + 17,))
    x = syn.bf16_bits_to_f32(big)
    assert abs(float(x.mean())) < 5e-3 and abs(float(x.std()) - 1.0) < 5e-3


def test_workload_shapes_and_ranges():
    wl = syn.CONFIGS["cfg2"]
    lens = syn.prefix_lengths(wl)
    assert lens.shape == (32,) and lens.min() >= 512 and lens.max() <= 4096
    assert np.array_equal(lens, syn.prefix_lengths(syn.CONFIGS["cfg2_d4"]))   # same pool, two block sizes
    n, mpps = syn.pages_needed(wl, lens)
    perm = syn.free_list_permutation(wl, n)
    assert sorted(perm.tolist()) == list(range(n))
    assert mpps * 64 >= lens.max() + wl.block
    assert syn.lm_head_bytes(wl) == 622329856
    assert syn.lm_head_bytes(syn.CONFIGS["cfg3"]) == 1557135360


def test_planted_hidden_states_spread_confidence_across_tau():
    wl = syn.CONFIGS["cfg0"].with_(batch=64)
    w = syn.lm_head_weight(wl)
    x = syn.block_inputs(wl, w)
    assert x.hidden.shape == (64, 4, 256) and x.q.shape == (64, 4, 4, 64) and x.k_blk.shape == (64, 4, 2, 64)
    h = syn.bf16_bits_to_f32(x.hidden).astype(np.float64).reshape(-1, 256)
    z = h @ syn.bf16_bits_to_f32(w).astype(np.float64).T
    p = np.exp(z - z.max(-1, keepdims=True)); p /= p.sum(-1, keepdims=True)
    top = p.max(-1)
    frac = float((top >= 0.9).mean())
    assert 0.25 < frac < 0.75                       # roughly half the positions clear tau = 0.9
    hit = (z.argmax(-1) == x.target.reshape(-1))
    assert hit[top >= 0.9].all()                     # a confident position is confident in the planted token
    y = syn.block_inputs(wl, w, step=1)
    assert not np.array_equal(x.hidden, y.hidden)
