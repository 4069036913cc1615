"""Test helpers that build the oracle's view of a synthetic workload and compare results."""
from __future__ import annotations

import numpy as np

from oracle import sdlm_oracle as orc
import sdlm_synth as syn

TOL_ATTN = 2e-2       # max-abs, bf16 attention outputs (fp32 accumulate)
TOL_CONF = 1e-3       # absolute, confidences
TOL_ENTROPY = 2e-3    # absolute, entropy in nats
GAP_FLAG = 1e-3       # tokens may differ only where the oracle's top-2 logit gap is below this
TAU_FLAG = 1e-4       # gamma may differ only where a running product is this close to tau


def oracle_cache(wl: syn.Workload, lengths, num_pages, mpps, prefix=None):
    s = wl.shape
    cache = orc.PagedKVCache(num_pages, s.page_size, s.n_kv_heads, s.head_dim, wl.batch, mpps,
                             syn.free_list_permutation(wl, num_pages))
    for b in range(wl.batch):
        k, v = prefix[b] if prefix else syn.prefix_kv(wl, b, int(lengths[b]))
        cache.add_sequence_fast(b, k, v)
    return cache


def bf16_bits_to_f64(bits):
    return orc.widen(bits)


def check_tokens(gpu_token, stats, report):
    """Bit-exact argmax except where the oracle's top-2 logits are nearly tied (reported)."""
    gpu = np.asarray(gpu_token).reshape(-1)
    bad = np.nonzero(gpu != stats.token)[0]
    for r in bad:
        assert stats.top2_gap[r] < GAP_FLAG, f"token mismatch at row {r}: gpu {gpu[r]} oracle {stats.token[r]} gap {stats.top2_gap[r]}"
        report.append(("token", int(r), int(gpu[r]), int(stats.token[r]), float(stats.top2_gap[r])))
    return len(bad)


def check_confidences(gpu_p, gpu_ent, stats):
    p = np.asarray(gpu_p, dtype=np.float64).reshape(-1)
    e = np.asarray(gpu_ent, dtype=np.float64).reshape(-1)
    dp = np.max(np.abs(p - stats.p_top1))
    de = np.max(np.abs(e - stats.entropy))
    V = None
    assert dp <= TOL_CONF, f"p_top1 max abs err {dp}"
    assert de <= TOL_ENTROPY, f"entropy max abs err {de}"
    return dp, de


def check_gamma(gpu_acc, commit, report):
    gpu = np.asarray(gpu_acc).reshape(-1)
    bad = np.nonzero(gpu != commit.accepted_len)[0]
    for b in bad:
        assert commit.tau_margin[b] < TAU_FLAG, f"gamma mismatch at seq {b}: gpu {gpu[b]} oracle {commit.accepted_len[b]} margin {commit.tau_margin[b]}"
        report.append(("gamma", int(b), int(gpu[b]), int(commit.accepted_len[b]), float(commit.tau_margin[b])))
    return len(bad)


def check_attention(gpu_bits, ref64):
    got = bf16_bits_to_f64(gpu_bits).reshape(ref64.shape)
    err = float(np.max(np.abs(got - ref64))) if ref64.size else 0.0
    assert np.all(np.isfinite(got)), "non-finite attention output"
    assert err <= TOL_ATTN, f"attention max abs err {err}"
    return err
