"""Puts a synthetic workload (sdlm_synth) on the device behind one library context.

Used by the tests, the benchmark and the smoke check to build identical device state.  It draws
inputs and marshals them; every step of the decode path itself runs in the library.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import numpy as np
import torch

import sdlm_synth as syn

from .binding import CONF_LOGIT, Sdlm, SdlmConfig, accept_commit_layers, bf16_tensor_from_bits


@dataclass
class DeviceBlock:
    q: torch.Tensor
    k_blk: torch.Tensor
    v_blk: torch.Tensor
    hidden: torch.Tensor
    host: syn.BlockInputs


@dataclass
class DeviceVerify:
    q: torch.Tensor        # [B, D, Hq, d]
    k_blk: torch.Tensor    # [B, 2D, Hkv, d]: real tokens' keys, then the [m] keys
    v_blk: torch.Tensor
    hidden: torch.Tensor   # [B, D, H]
    host: "syn.VerifyInputs"
    host_hidden: np.ndarray


@dataclass
class StepOutputs:
    attn: torch.Tensor
    token: torch.Tensor
    p_top1: torch.Tensor
    entropy: torch.Tensor
    accepted_len: torch.Tensor
    out_tokens: torch.Tensor


class DeviceProblem:
    def __init__(self, wl: syn.Workload, w_bits: Optional[np.ndarray] = None, lengths: Optional[np.ndarray] = None,
                 max_block: Optional[int] = None, keep_prefix: bool = True, prefix=None, fill: bool = True):
        """prefix: the per-sequence (k, v) bit arrays to use instead of drawing them again; fill=False
        leaves the cache empty (tables reset, no sequence added)."""
        self.wl = wl
        s = wl.shape
        self.lengths = syn.prefix_lengths(wl) if lengths is None else np.asarray(lengths, dtype=np.int32)
        self.num_pages, self.mpps = syn.pages_needed(wl, self.lengths)
        self.free_list = syn.free_list_permutation(wl, self.num_pages)
        self.cfg = SdlmConfig(s.n_q_heads, s.n_kv_heads, s.head_dim, s.hidden, s.vocab, self.num_pages, wl.batch,
                              self.mpps, max_block=max_block or wl.block, page_size=s.page_size)
        self.sd = Sdlm(self.cfg)
        self.w_bits = syn.lm_head_weight(wl) if w_bits is None else w_bits
        self.w_lm = bf16_tensor_from_bits(self.w_bits)
        self.prefix = list(prefix) if prefix is not None else []
        if fill:
            self.reset_cache(keep_prefix)
        else:
            self.sd.kv_reset(self.free_list)

    def reset_cache(self, keep_prefix: bool = True) -> None:
        """Free list := the seeded permutation, then every sequence's prefix is added in slot order."""
        self.sd.kv_reset(self.free_list)
        regenerate = not self.prefix
        for b in range(self.wl.batch):
            if regenerate:
                k, v = syn.prefix_kv(self.wl, b, int(self.lengths[b]))
                if keep_prefix:
                    self.prefix.append((k, v))
            else:
                k, v = self.prefix[b]
            if k.shape[0] > 0:
                self.sd.kv_add_seq(b, bf16_tensor_from_bits(k), bf16_tensor_from_bits(v))
        torch.cuda.synchronize()

    def block(self, step: int = 0) -> DeviceBlock:
        x = syn.block_inputs(self.wl, self.w_bits, step)
        return DeviceBlock(bf16_tensor_from_bits(x.q), bf16_tensor_from_bits(x.k_blk), bf16_tensor_from_bits(x.v_blk),
                           bf16_tensor_from_bits(x.hidden), x)

    def verify_block(self, step: int = 0, p_agree: float = 0.8) -> "DeviceVerify":
        """Device copies of the verification pass's inputs of step `step` (self-speculative decoding)."""
        wl = self.wl
        v = syn.verify_inputs(wl, self.w_bits, step)
        h = syn.verify_hidden(wl, self.w_bits, step, p_agree)
        return DeviceVerify(bf16_tensor_from_bits(v.q), bf16_tensor_from_bits(v.k_blk), bf16_tensor_from_bits(v.v_blk),
                            bf16_tensor_from_bits(h), v, h)

    def speculative_step(self, x: DeviceBlock, xv: "DeviceVerify", out: StepOutputs, out_v: StepOutputs,
                         stream=None) -> None:
        """One self-speculative step (Sec. 3.4) on device-resident inputs, five library calls: first pass
        (attention, LM head -> speculative tokens), verification pass (attention over the real
        tokens' and the [m] keys under the verification inputs' visibility, LM head -> verification tokens), then gamma_verify and the commit of
        the kept real-token rows.  No host synchronisation."""
        sd = self.sd
        sd.block_attn(x.q, x.k_blk, x.v_blk, out.attn, stream=stream)
        sd.lmhead_confidence(x.hidden, self.w_lm, out.token, out.p_top1, out.entropy, stream=stream)
        sd.block_attn_verify(xv.q, xv.k_blk, xv.v_blk, out_v.attn, stream=stream)
        sd.lmhead_confidence(xv.hidden, self.w_lm, out_v.token, out_v.p_top1, out_v.entropy, stream=stream)
        sd.verify_commit(out.token, out_v.token, x.k_blk, x.v_blk, out.accepted_len, out.out_tokens, stream=stream)

    def alloc_outputs(self) -> StepOutputs:
        wl, s, dev = self.wl, self.wl.shape, self.sd.device
        B, D = wl.batch, wl.block
        return StepOutputs(torch.empty((B, D, s.n_q_heads, s.head_dim), dtype=torch.bfloat16, device=dev),
                           torch.empty((B, D), dtype=torch.int32, device=dev),
                           torch.empty((B, D), dtype=torch.float32, device=dev),
                           torch.empty((B, D), dtype=torch.float32, device=dev),
                           torch.empty(B, dtype=torch.int32, device=dev),
                           torch.empty((B, D), dtype=torch.int32, device=dev))

    def step(self, x: DeviceBlock, tau: float, out: Optional[StepOutputs] = None, mode: int = CONF_LOGIT,
             stream=None, fused: bool = False) -> StepOutputs:
        """(a) + (b) + (c) on device-resident inputs: three library calls, no host synchronisation."""
        out = out or self.alloc_outputs()
        sd = self.sd
        if fused:
            sd.decode_step(tau, x.q, x.k_blk, x.v_blk, x.hidden, self.w_lm, out.attn, out.token, out.p_top1, out.entropy,
                           out.accepted_len, out.out_tokens, mode=mode, stream=stream)
            return out
        sd.block_attn(x.q, x.k_blk, x.v_blk, out.attn, stream=stream)
        sd.lmhead_confidence(x.hidden, self.w_lm, out.token, out.p_top1, out.entropy, stream=stream)
        sd.accept_commit(tau, out.token, out.p_top1, out.entropy, x.k_blk, x.v_blk, mode, out.accepted_len,
                         out.out_tokens, stream=stream)
        return out


# ---- a stack of decoder layers around the path (Qwen-2.5 shape) -------------------------------------
@dataclass
class LayerWeights:
    ln1: torch.Tensor    # [H]
    wq: torch.Tensor     # [Hq*d, H]
    bq: torch.Tensor     # [Hq*d]
    wk: torch.Tensor     # [Hkv*d, H]
    bk: torch.Tensor
    wv: torch.Tensor
    bv: torch.Tensor
    wo: torch.Tensor     # [H, Hq*d]
    ln2: torch.Tensor    # [H]
    wgu: torch.Tensor    # [2I, H]: gate rows, then up rows
    wdown: torch.Tensor  # [H, I]


class DecoderStack:
    """n_layers pre-norm decoder layers (RMSNorm, biased q/k/v projections, rotary positions, block
    attention over that layer's own paged cache, output projection, SwiGLU MLP), a final RMSNorm and the
    LM head with acceptance: one whole-model NSP decode step, every operation a library call.  Every
    layer has its own context (KV pool and tables); all tables move in lockstep because every layer
    commits the same accepted lengths."""

    EPS = 1e-6
    THETA = 1.0e6

    def __init__(self, wl: syn.Workload, n_layers: int, intermediate: int, lengths: np.ndarray, layers, ln_f, w_lm,
                 prefix_fn, drop_split_weights: bool = False):
        """layers: list of LayerWeights; prefix_fn(layer, b, length) -> (k, v) device tensors [length, Hkv, d].
        drop_split_weights: forget every layer's wq / wk / wv / wgu once the stacked and interleaved copies that
        the step reads exist (a 32B-shaped stack does not fit twice)."""
        s = wl.shape
        self.wl, self.L, self.I = wl, n_layers, intermediate
        self.lengths = np.asarray(lengths, dtype=np.int32)
        self.num_pages, self.mpps = syn.pages_needed(wl, self.lengths)
        self.free_list = syn.free_list_permutation(wl, self.num_pages)
        cfg = SdlmConfig(s.n_q_heads, s.n_kv_heads, s.head_dim, s.hidden, s.vocab, self.num_pages, wl.batch, self.mpps,
                         max_block=wl.block, page_size=s.page_size)
        self.ctx = [Sdlm(cfg) for _ in range(n_layers)]
        self.layers, self.ln_f, self.w_lm = layers, ln_f, w_lm
        w0 = layers[0]
        self._weight_bytes = n_layers * sum(t.numel() * 2 for t in (w0.wq, w0.wk, w0.wv, w0.wo, w0.wgu, w0.wdown)) + w_lm.numel() * 2
        self.wqkv, self.bqkv, self.wgu_il = [], [], []
        for w in layers:
            # q, k and v come from one product over the stacked weight
            self.wqkv.append(torch.cat([w.wq, w.wk, w.wv], dim=0).contiguous())
            self.bqkv.append(torch.cat([w.bq, w.bk, w.bv], dim=0).contiguous())
            # gate and up rows interleaved, so that the product's epilogue can gate in registers
            self.wgu_il.append(torch.stack([w.wgu[:intermediate], w.wgu[intermediate:]], dim=1).reshape(2 * intermediate, -1).contiguous())
            if drop_split_weights:
                w.wq = w.wk = w.wv = w.wgu = None
        for l, sd in enumerate(self.ctx):
            sd.kv_reset(self.free_list)
            for b in range(wl.batch):
                if self.lengths[b] > 0:
                    k, v = prefix_fn(l, b, int(self.lengths[b]))
                    sd.kv_add_seq(b, k, v)
        dev = self.ctx[0].device
        B, D, rows = wl.batch, wl.block, wl.batch * wl.block
        e = lambda *shape: torch.empty(shape, dtype=torch.bfloat16, device=dev)
        self.h, self.x = e(rows, s.hidden), e(rows, s.hidden)
        self.q, self.attn = e(B, D, s.n_q_heads, s.head_dim), e(B, D, s.n_q_heads, s.head_dim)
        self.k = [e(B, D, s.n_kv_heads, s.head_dim) for _ in range(n_layers)]
        self.v = [e(B, D, s.n_kv_heads, s.head_dim) for _ in range(n_layers)]
        self.gu, self.act = e(rows, 2 * intermediate), e(rows, intermediate)
        self.saved = [sd.kv_save() for sd in self.ctx]
        torch.cuda.synchronize()

    def restore(self, stream=None) -> None:
        for sd, sv in zip(self.ctx, self.saved):
            sd.kv_restore(sv, stream=stream)

    def step(self, h0: torch.Tensor, tau: float, out: StepOutputs, stream=None) -> None:
        """h0 [B, D, H]: the block's input embeddings.  out.attn is not used (attention is per layer)."""
        wl, s = self.wl, self.wl.shape
        self.h.copy_(h0.reshape(self.h.shape))
        self.ctx[0].rmsnorm(self.h, self.layers[0].ln1, self.EPS, self.x, stream=stream)
        for l, (sd, w) in enumerate(zip(self.ctx, self.layers)):
            sd.linear3_rope(self.x, self.wqkv[l], self.bqkv[l], self.q, self.k[l], self.v[l], self.THETA, stream=stream)
            sd.block_attn(self.q, self.k[l], self.v[l], self.attn, stream=stream)
            # the residual stream is updated in place and its norm for the next product comes with it
            sd.linear_rmsnorm(self.attn, w.wo, w.ln2, self.EPS, None, self.h, self.h, self.x, stream=stream)
            sd.linear_swiglu(self.x, self.wgu_il[l], self.act, stream=stream)
            nxt = self.layers[l + 1].ln1 if l + 1 < self.L else self.ln_f
            sd.linear_rmsnorm(self.act, w.wdown, nxt, self.EPS, None, self.h, self.h, self.x, stream=stream)
        sd0 = self.ctx[0]
        sd0.lmhead_confidence(self.x, self.w_lm, out.token, out.p_top1, out.entropy, stream=stream)
        accept_commit_layers(self.ctx, tau, out.token, out.p_top1, out.entropy, self.k, self.v, out.accepted_len,
                             out.out_tokens, stream=stream)

    def launches(self) -> int:
        return sum(sd.launch_count() for sd in self.ctx)

    def weight_bytes(self) -> int:
        return self._weight_bytes
