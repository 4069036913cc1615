"""ctypes binding of libsdlm.so: argument marshalling only.

Every method has the name of the C entry point it calls (``sdlm_`` dropped) and does nothing but
check tensor types, hand raw device pointers to the library and raise on a non-zero status.  All
computation runs in the library's CUDA kernels; if the library cannot be loaded, or there is no
CUDA device, creating a context raises -- there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional, Sequence, Tuple

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsdlm.so")

CONF_LOGIT, CONF_ENTROPY = 0, 1
KV_RESET, KV_ADD_SEQ, KV_RELEASE_SEQ, KV_QUERY, KV_GATHER, KV_EXPORT, KV_IMPORT, KV_SAVE, KV_RESTORE = range(9)
OPT_LMHEAD_KERNEL = 0
OPT_STEP_OVERLAP = 1
OPT_ATTN_ITEM_COST = 2
OPT_ATTN_MIN_RANGE = 3
OPT_HOST_TWO_STREAMS = 4
OPT_ATTN_EARLY_PREFETCH = 5
OPT_HOST_HIDDEN_BY_ATTN = 6
OPT_HOST_INPLACE_MAX_KB = 7

STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "SHAPE", 3: "UNSUPPORTED", 4: "OUT_OF_PAGES", 5: "CUDA",
                6: "TIMEOUT", 7: "DEVICE_CHECK", 8: "WORKSPACE"}

EXPORTED = ["sdlm_pool_bytes", "sdlm_workspace_bytes", "sdlm_create", "sdlm_destroy", "sdlm_status_str",
            "sdlm_kv_pages", "sdlm_block_attn", "sdlm_lmhead_confidence", "sdlm_lmhead_confidence_static", "sdlm_accept_commit",
            "sdlm_device_status", "sdlm_decode_step", "sdlm_decode_step_host", "sdlm_set_option", "sdlm_launch_count",
            "sdlm_block_attn_masked", "sdlm_verify_commit", "sdlm_accept_commit_carry",
            "sdlm_block_attn_verify", "sdlm_block_attn_carry", "sdlm_causal_attn",
            "sdlm_linear", "sdlm_linear3", "sdlm_linear3_rope", "sdlm_rmsnorm", "sdlm_rope_block", "sdlm_swiglu", "sdlm_selftest_bounded_wait", "sdlm_rope_block2", "sdlm_accept_commit_layers", "sdlm_block_attn_prefix", "sdlm_linear_swiglu",
            "sdlm_block_attn_masked_prefix", "sdlm_linear_rmsnorm"]


def accept_commit_layers(contexts, tau: float, token, p_top1, entropy, k_blks, v_blks, accepted_len, out_tokens,
                         mode: int = 0, seq_ids=None, stream=None) -> None:
    """sdlm_accept_commit_layers: one launch commits the same accepted rows into every layer's cache."""
    sd0 = contexts[0]
    n = len(contexts)
    batch, D = int(k_blks[0].shape[0]), int(k_blks[0].shape[1])
    ctx_arr = (C.c_void_p * n)(*[c.ctx.value for c in contexts])
    k_arr = (C.c_void_p * n)(*[_ptr(_dev(t, torch.bfloat16, "k_blk")) for t in k_blks])
    v_arr = (C.c_void_p * n)(*[_ptr(_dev(t, torch.bfloat16, "v_blk")) for t in v_blks])
    sd0._check("sdlm_accept_commit_layers", sd0.lib.sdlm_accept_commit_layers(
        ctx_arr, n, batch, D, _ptr(seq_ids), float(tau), int(mode), _ptr(_dev(token, torch.int32, "token")),
        _ptr(_dev(p_top1, torch.float32, "p_top1")), _ptr(_dev(entropy, torch.float32, "entropy")), k_arr, v_arr,
        _ptr(_dev(accepted_len, torch.int32, "accepted_len")), _ptr(_dev(out_tokens, torch.int32, "out_tokens")),
        _stream_ptr(stream)))


class SdlmError(RuntimeError):
    def __init__(self, call: str, code: int, text: str):
        super().__init__(f"{call} failed: {STATUS_NAMES.get(code, code)} ({text})")
        self.code = code


class _Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_q_heads", "n_kv_heads", "head_dim", "hidden", "vocab", "page_size",
                                          "num_pages", "max_batch", "max_pages_per_seq", "max_block")] + \
               [("softmax_scale", C.c_float)]


class _KvArgs(C.Structure):
    _fields_ = [("seq", C.c_int32), ("length", C.c_int32), ("k", C.c_void_p), ("v", C.c_void_p),
                ("k_out", C.c_void_p), ("v_out", C.c_void_p), ("free_list", C.c_void_p),
                ("host_buf", C.c_void_p), ("host_bytes", C.c_size_t), ("dev_buf", C.c_void_p),
                ("dev_bytes", C.c_size_t)]


class _KvResult(C.Structure):
    _fields_ = [("page_table", C.c_void_p), ("seq_len", C.c_void_p), ("free_list", C.c_void_p),
                ("free_head", C.c_void_p), ("free_tail", C.c_void_p), ("device_status", C.c_void_p),
                ("table_bytes", C.c_size_t)]


@dataclass
class SdlmConfig:
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    hidden: int
    vocab: int
    num_pages: int
    max_batch: int
    max_pages_per_seq: int
    max_block: int = 8
    page_size: int = 64
    softmax_scale: float = 0.0

    def to_c(self) -> _Config:
        return _Config(self.n_q_heads, self.n_kv_heads, self.head_dim, self.hidden, self.vocab, self.page_size,
                       self.num_pages, self.max_batch, self.max_pages_per_seq, self.max_block, self.softmax_scale)


_lib = None


def load_library(path: Optional[str] = None) -> C.CDLL:
    """Loads libsdlm.so and declares the signatures of include/sdlm.h."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    path = path or LIB_PATH
    if not os.path.exists(path):
        raise SdlmError("load_library", 5, f"{path} not built; run paper_2509_24007_b200/build.py")
    lib = C.CDLL(path)
    vp, i32, f32 = C.c_void_p, C.c_int32, C.c_float
    lib.sdlm_pool_bytes.restype = C.c_size_t
    lib.sdlm_pool_bytes.argtypes = [C.POINTER(_Config)]
    lib.sdlm_workspace_bytes.restype = C.c_size_t
    lib.sdlm_workspace_bytes.argtypes = [C.POINTER(_Config)]
    lib.sdlm_create.restype = C.c_int
    lib.sdlm_create.argtypes = [C.POINTER(_Config), vp, C.c_size_t, vp, C.c_size_t, C.POINTER(vp)]
    lib.sdlm_destroy.restype = None
    lib.sdlm_destroy.argtypes = [vp]
    lib.sdlm_status_str.restype = C.c_char_p
    lib.sdlm_status_str.argtypes = [C.c_int]
    lib.sdlm_kv_pages.restype = C.c_int
    lib.sdlm_kv_pages.argtypes = [vp, C.c_int, C.POINTER(_KvArgs), C.POINTER(_KvResult), vp]
    lib.sdlm_block_attn.restype = C.c_int
    lib.sdlm_block_attn.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp]
    lib.sdlm_lmhead_confidence.restype = C.c_int
    lib.sdlm_lmhead_confidence.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.sdlm_lmhead_confidence_static.restype = C.c_int
    lib.sdlm_lmhead_confidence_static.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.sdlm_block_attn_prefix.restype = C.c_int
    lib.sdlm_block_attn_prefix.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp, vp]
    lib.sdlm_block_attn_masked.restype = C.c_int
    lib.sdlm_block_attn_masked.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp]
    lib.sdlm_block_attn_masked_prefix.restype = C.c_int
    lib.sdlm_block_attn_masked_prefix.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.sdlm_accept_commit_carry.restype = C.c_int
    lib.sdlm_accept_commit_carry.argtypes = [vp, i32, i32, i32, vp, vp, f32, C.c_int, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.sdlm_causal_attn.restype = C.c_int
    lib.sdlm_causal_attn.argtypes = [vp, i32, i32, i32, vp, vp, vp]
    lib.sdlm_block_attn_verify.restype = C.c_int
    lib.sdlm_block_attn_verify.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp]
    lib.sdlm_block_attn_carry.restype = C.c_int
    lib.sdlm_block_attn_carry.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp]
    lib.sdlm_linear_rmsnorm.restype = C.c_int
    lib.sdlm_linear_rmsnorm.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp, vp, f32, vp, vp]
    lib.sdlm_linear.restype = C.c_int
    lib.sdlm_linear.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp, vp]
    lib.sdlm_selftest_bounded_wait.restype = C.c_int
    lib.sdlm_selftest_bounded_wait.argtypes = [vp, vp]
    lib.sdlm_linear_swiglu.restype = C.c_int
    lib.sdlm_linear_swiglu.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp]
    lib.sdlm_linear3.restype = C.c_int
    lib.sdlm_linear3.argtypes = [vp, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp]
    lib.sdlm_linear3_rope.restype = C.c_int
    lib.sdlm_linear3_rope.argtypes = [vp, i32, i32, vp, i32, i32, i32, vp, vp, vp, vp, vp, vp, f32, vp]
    lib.sdlm_rmsnorm.restype = C.c_int
    lib.sdlm_rmsnorm.argtypes = [vp, i32, i32, vp, vp, f32, vp, vp]
    lib.sdlm_rope_block.restype = C.c_int
    lib.sdlm_rope_block.argtypes = [vp, i32, i32, vp, i32, vp, f32, vp]
    lib.sdlm_accept_commit_layers.restype = C.c_int
    lib.sdlm_accept_commit_layers.argtypes = [vp, i32, i32, i32, vp, f32, C.c_int, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.sdlm_rope_block2.restype = C.c_int
    lib.sdlm_rope_block2.argtypes = [vp, i32, i32, vp, i32, vp, i32, vp, f32, vp]
    lib.sdlm_swiglu.restype = C.c_int
    lib.sdlm_swiglu.argtypes = [vp, i32, i32, vp, vp, vp]
    lib.sdlm_verify_commit.restype = C.c_int
    lib.sdlm_verify_commit.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.sdlm_accept_commit.restype = C.c_int
    lib.sdlm_accept_commit.argtypes = [vp, i32, i32, vp, f32, C.c_int, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.sdlm_device_status.restype = C.c_int
    lib.sdlm_device_status.argtypes = [vp, vp, i32, vp]
    lib.sdlm_decode_step.restype = C.c_int
    lib.sdlm_decode_step.argtypes = [vp, i32, i32, vp, f32, C.c_int] + [vp] * 12
    lib.sdlm_decode_step_host.restype = C.c_int
    lib.sdlm_decode_step_host.argtypes = [vp, i32, i32, vp, f32, C.c_int] + [vp] * 12
    lib.sdlm_set_option.restype = C.c_int
    lib.sdlm_set_option.argtypes = [vp, C.c_int, i32]
    lib.sdlm_launch_count.restype = C.c_uint64
    lib.sdlm_launch_count.argtypes = [vp]
    if path == LIB_PATH:
        _lib = lib
    return lib


def bf16_tensor_from_bits(bits: np.ndarray, device="cuda") -> torch.Tensor:
    """numpy uint16 bf16 bit patterns -> torch.bfloat16 tensor with the same bits."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).to(device)


def bits_from_bf16_tensor(t: torch.Tensor) -> np.ndarray:
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _dev(t: torch.Tensor, dtype, name: str) -> torch.Tensor:
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{name}: expected a contiguous CUDA tensor of {dtype}")
    return t


def _host(t: torch.Tensor, dtype, name: str) -> torch.Tensor:
    if not (isinstance(t, torch.Tensor) and not t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{name}: expected a contiguous host tensor of {dtype}")
    return t


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    return (stream or torch.cuda.current_stream()).cuda_stream


class Sdlm:
    """One library context over torch-allocated device memory (KV pool + workspace)."""

    def __init__(self, cfg: SdlmConfig, device: Optional[int] = None):
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise SdlmError("sdlm_create", 5, "no CUDA device: the library has no CPU path")
        self.cfg = cfg
        self.device = torch.device("cuda", torch.cuda.current_device() if device is None else device)
        c = cfg.to_c()
        pool_bytes = self.lib.sdlm_pool_bytes(C.byref(c))
        ws_bytes = self.lib.sdlm_workspace_bytes(C.byref(c))
        if pool_bytes == 0 or ws_bytes == 0:
            raise SdlmError("sdlm_pool_bytes", 3, "configuration rejected")
        with torch.cuda.device(self.device):
            self._pool = torch.empty(pool_bytes + 1024, dtype=torch.uint8, device=self.device)
            self._ws = torch.empty(ws_bytes + 256, dtype=torch.uint8, device=self.device)
            pool_ptr = (self._pool.data_ptr() + 1023) // 1024 * 1024
            ws_ptr = (self._ws.data_ptr() + 255) // 256 * 256
            out = C.c_void_p()
            self._check("sdlm_create", self.lib.sdlm_create(C.byref(c), pool_ptr, pool_bytes, ws_ptr, ws_bytes,
                                                            C.byref(out)))
        self.ctx = out
        self.pool_bytes, self.workspace_bytes = pool_bytes, ws_bytes

    def close(self) -> None:
        if getattr(self, "ctx", None):
            self.lib.sdlm_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, call: str, code: int) -> None:
        if code != 0:
            raise SdlmError(call, code, self.lib.sdlm_status_str(code).decode())

    # ---- sdlm_kv_pages -------------------------------------------------------------------
    def kv_pages(self, op: int, seq: int = 0, length: int = 0, k: Optional[torch.Tensor] = None,
                 v: Optional[torch.Tensor] = None, k_out: Optional[torch.Tensor] = None,
                 v_out: Optional[torch.Tensor] = None, free_list: Optional[np.ndarray] = None,
                 host_buf: Optional[np.ndarray] = None, dev_buf: Optional[torch.Tensor] = None, stream=None) -> _KvResult:
        a = _KvArgs()
        a.seq, a.length = seq, length
        keep = []
        if k is not None:
            a.k, a.v = _ptr(_dev(k, torch.bfloat16, "k")), _ptr(_dev(v, torch.bfloat16, "v"))
        if k_out is not None:
            a.k_out, a.v_out = _ptr(_dev(k_out, torch.bfloat16, "k_out")), _ptr(_dev(v_out, torch.bfloat16, "v_out"))
        if free_list is not None:
            fl = np.ascontiguousarray(free_list, dtype=np.int32)
            if fl.shape != (self.cfg.num_pages,):
                raise TypeError("free_list: expected int32[num_pages]")
            keep.append(fl)
            a.free_list = fl.ctypes.data
        if host_buf is not None:
            a.host_buf, a.host_bytes = host_buf.ctypes.data, host_buf.nbytes
        if dev_buf is not None:
            _dev(dev_buf, torch.uint8, "dev_buf")
            a.dev_buf, a.dev_bytes = dev_buf.data_ptr(), dev_buf.numel()
        r = _KvResult()
        self._check("sdlm_kv_pages", self.lib.sdlm_kv_pages(self.ctx, op, C.byref(a), C.byref(r), _stream_ptr(stream)))
        return r

    def kv_reset(self, free_list: Optional[np.ndarray] = None, stream=None) -> None:
        self.kv_pages(KV_RESET, free_list=free_list, stream=stream)

    def kv_add_seq(self, seq: int, k: torch.Tensor, v: torch.Tensor, stream=None) -> None:
        self.kv_pages(KV_ADD_SEQ, seq=seq, length=int(k.shape[0]), k=k, v=v, stream=stream)

    def kv_release_seq(self, seq: int, stream=None) -> None:
        self.kv_pages(KV_RELEASE_SEQ, seq=seq, stream=stream)

    def kv_gather(self, seq: int, length: int, stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
        shp = (length, self.cfg.n_kv_heads, self.cfg.head_dim)
        k = torch.zeros(shp, dtype=torch.bfloat16, device=self.device)
        v = torch.zeros(shp, dtype=torch.bfloat16, device=self.device)
        self.kv_pages(KV_GATHER, seq=seq, length=length, k_out=k, v_out=v, stream=stream)
        return k, v

    def kv_tables(self) -> dict:
        """Host copies of the live tables (synchronises the current stream)."""
        r = self.kv_pages(KV_QUERY)
        buf = np.empty(r.table_bytes, dtype=np.uint8)
        self.kv_pages(KV_EXPORT, host_buf=buf)
        return self._parse_tables(buf)

    def _parse_tables(self, buf: np.ndarray) -> dict:
        cfg = self.cfg
        al = lambda x: (x + 255) // 256 * 256
        off = 0
        hdr = buf[off:off + 64].view(np.int32); off = al(off + 64)
        n = cfg.max_batch * cfg.max_pages_per_seq * 4
        pt = buf[off:off + n].view(np.int32).reshape(cfg.max_batch, cfg.max_pages_per_seq); off = al(off + n)
        sl = buf[off:off + cfg.max_batch * 4].view(np.int32); off = al(off + cfg.max_batch * 4)
        fl = buf[off:off + cfg.num_pages * 4].view(np.int32)
        return {"status": hdr[:4].copy(), "free_head": int(hdr.view(np.uint32)[4]), "free_tail": int(hdr.view(np.uint32)[5]),
                "page_table": pt.copy(), "seq_len": sl.copy(), "free_list": fl.copy()}

    def kv_export(self) -> np.ndarray:
        r = self.kv_pages(KV_QUERY)
        buf = np.empty(r.table_bytes, dtype=np.uint8)
        self.kv_pages(KV_EXPORT, host_buf=buf)
        return buf

    def copy_pool_from(self, other: "Sdlm", stream=None) -> None:
        """Raw copy of another context's KV pool (same configuration) into this one's, for resuming from
        exported tables."""
        if other.pool_bytes != self.pool_bytes:
            raise ValueError("pools differ in size")
        a = (self._pool.data_ptr() + 1023) // 1024 * 1024 - self._pool.data_ptr()
        b = (other._pool.data_ptr() + 1023) // 1024 * 1024 - other._pool.data_ptr()
        with torch.cuda.stream(stream or torch.cuda.current_stream()):
            self._pool[a:a + self.pool_bytes].copy_(other._pool[b:b + other.pool_bytes])

    def kv_save(self, dev_buf: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        """Device-side snapshot of the tables (no host synchronisation); returns the buffer."""
        if dev_buf is None:
            dev_buf = torch.empty(self.kv_pages(KV_QUERY).table_bytes, dtype=torch.uint8, device=self.device)
        self.kv_pages(KV_SAVE, dev_buf=dev_buf, stream=stream)
        return dev_buf

    def kv_restore(self, dev_buf: torch.Tensor, stream=None) -> None:
        self.kv_pages(KV_RESTORE, dev_buf=dev_buf, stream=stream)

    def kv_import(self, buf: np.ndarray) -> None:
        self.kv_pages(KV_IMPORT, host_buf=np.ascontiguousarray(buf))

    # ---- the three hot-path calls --------------------------------------------------------
    def block_attn(self, q: torch.Tensor, k_blk: torch.Tensor, v_blk: torch.Tensor, out: Optional[torch.Tensor] = None,
                   seq_ids: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        batch, D = int(q.shape[0]), int(q.shape[1])
        _dev(q, torch.bfloat16, "q"); _dev(k_blk, torch.bfloat16, "k_blk"); _dev(v_blk, torch.bfloat16, "v_blk")
        if out is None:
            out = torch.empty_like(q)
        if seq_ids is not None:
            _dev(seq_ids, torch.int32, "seq_ids")
        self._check("sdlm_block_attn", self.lib.sdlm_block_attn(self.ctx, batch, D, _ptr(seq_ids), _ptr(q), _ptr(k_blk),
                                                                _ptr(v_blk), _ptr(_dev(out, torch.bfloat16, "out")),
                                                                _stream_ptr(stream)))
        return out

    def block_attn_prefix(self, q: torch.Tensor, k_blk: torch.Tensor, v_blk: torch.Tensor, seq_ids: torch.Tensor,
                          prefix_len: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        """sdlm_block_attn_prefix: row b sees the first prefix_len[b] cached tokens of slot seq_ids[b]."""
        batch, D = int(q.shape[0]), int(q.shape[1])
        _dev(q, torch.bfloat16, "q"); _dev(k_blk, torch.bfloat16, "k_blk"); _dev(v_blk, torch.bfloat16, "v_blk")
        _dev(seq_ids, torch.int32, "seq_ids"); _dev(prefix_len, torch.int32, "prefix_len")
        if out is None:
            out = torch.empty_like(q)
        self._check("sdlm_block_attn_prefix", self.lib.sdlm_block_attn_prefix(
            self.ctx, batch, D, _ptr(seq_ids), _ptr(prefix_len), _ptr(q), _ptr(k_blk), _ptr(v_blk),
            _ptr(_dev(out, torch.bfloat16, "out")), _stream_ptr(stream)))
        return out

    def block_attn_masked(self, q: torch.Tensor, k_blk: torch.Tensor, v_blk: torch.Tensor, vis: torch.Tensor,
                          out: Optional[torch.Tensor] = None, seq_ids: Optional[torch.Tensor] = None,
                          stream=None) -> torch.Tensor:
        """sdlm_block_attn_masked: vis [batch, n_q] int32 holds the uint32 visibility words."""
        batch, n_q, n_k = int(q.shape[0]), int(q.shape[1]), int(k_blk.shape[1])
        _dev(q, torch.bfloat16, "q"); _dev(k_blk, torch.bfloat16, "k_blk"); _dev(v_blk, torch.bfloat16, "v_blk")
        _dev(vis, torch.int32, "vis")
        if tuple(vis.shape) != (batch, n_q):
            raise ValueError("vis must be [batch, n_q]")
        if out is None:
            out = torch.empty_like(q)
        if seq_ids is not None:
            _dev(seq_ids, torch.int32, "seq_ids")
        self._check("sdlm_block_attn_masked", self.lib.sdlm_block_attn_masked(
            self.ctx, batch, n_q, n_k, _ptr(seq_ids), _ptr(q), _ptr(k_blk), _ptr(v_blk), _ptr(vis),
            _ptr(_dev(out, torch.bfloat16, "out")), _stream_ptr(stream)))
        return out

    def causal_attn(self, seq: int, q: torch.Tensor, first_pos: int = 0, out: Optional[torch.Tensor] = None,
                    stream=None) -> torch.Tensor:
        """sdlm_causal_attn: q [n_rows, Hq, d]; row r attends to the cached tokens 0 .. first_pos + r of slot seq."""
        _dev(q, torch.bfloat16, "q")
        if out is None:
            out = torch.empty_like(q)
        self._check("sdlm_causal_attn", self.lib.sdlm_causal_attn(
            self.ctx, int(seq), int(first_pos), int(q.shape[0]), _ptr(q), _ptr(_dev(out, torch.bfloat16, "out")),
            _stream_ptr(stream)))
        return out

    def block_attn_verify(self, q: torch.Tensor, k_blk: torch.Tensor, v_blk: torch.Tensor,
                          out: Optional[torch.Tensor] = None, seq_ids: Optional[torch.Tensor] = None,
                          stream=None) -> torch.Tensor:
        """sdlm_block_attn_verify: q [batch, D, Hq, d], k_blk / v_blk [batch, 2D, Hkv, d] (real tokens, then masks)."""
        batch, D = int(q.shape[0]), int(q.shape[1])
        _dev(q, torch.bfloat16, "q"); _dev(k_blk, torch.bfloat16, "k_blk"); _dev(v_blk, torch.bfloat16, "v_blk")
        if int(k_blk.shape[1]) != 2 * D or int(v_blk.shape[1]) != 2 * D:
            raise ValueError("k_blk / v_blk must hold 2D rows per sequence")
        if out is None:
            out = torch.empty_like(q)
        if seq_ids is not None:
            _dev(seq_ids, torch.int32, "seq_ids")
        self._check("sdlm_block_attn_verify", self.lib.sdlm_block_attn_verify(
            self.ctx, batch, D, _ptr(seq_ids), _ptr(q), _ptr(k_blk), _ptr(v_blk),
            _ptr(_dev(out, torch.bfloat16, "out")), _stream_ptr(stream)))
        return out

    def block_attn_carry(self, q: torch.Tensor, k_rows: torch.Tensor, v_rows: torch.Tensor, carry_len: torch.Tensor,
                         c_max: int, out: Optional[torch.Tensor] = None, seq_ids: Optional[torch.Tensor] = None,
                         stream=None) -> torch.Tensor:
        """sdlm_block_attn_carry: q [batch, c_max + D, Hq, d], k_rows / v_rows [batch, c_max + D, Hkv, d],
        carry_len [batch] int32 on the device."""
        batch, R = int(q.shape[0]), int(q.shape[1])
        _dev(q, torch.bfloat16, "q"); _dev(k_rows, torch.bfloat16, "k_rows"); _dev(v_rows, torch.bfloat16, "v_rows")
        _dev(carry_len, torch.int32, "carry_len")
        if int(k_rows.shape[1]) != R or int(v_rows.shape[1]) != R or carry_len.numel() != batch or not 0 <= c_max < R:
            raise ValueError("q, k_rows, v_rows must hold c_max + D rows per sequence and carry_len one entry each")
        if out is None:
            out = torch.empty_like(q)
        if seq_ids is not None:
            _dev(seq_ids, torch.int32, "seq_ids")
        self._check("sdlm_block_attn_carry", self.lib.sdlm_block_attn_carry(
            self.ctx, batch, R - int(c_max), int(c_max), _ptr(seq_ids), _ptr(carry_len), _ptr(q), _ptr(k_rows),
            _ptr(v_rows), _ptr(_dev(out, torch.bfloat16, "out")), _stream_ptr(stream)))
        return out

    def block_attn_masked_prefix(self, q: torch.Tensor, k_blk: torch.Tensor, v_blk: torch.Tensor, vis: torch.Tensor,
                                 seq_ids: torch.Tensor, prefix_len: torch.Tensor,
                                 out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        """sdlm_block_attn_masked_prefix: vis [batch, n_q] int32 words, seq_ids and prefix_len [batch] int32."""
        batch, n_q, n_k = int(q.shape[0]), int(q.shape[1]), int(k_blk.shape[1])
        _dev(q, torch.bfloat16, "q"); _dev(k_blk, torch.bfloat16, "k_blk"); _dev(v_blk, torch.bfloat16, "v_blk")
        _dev(vis, torch.int32, "vis"); _dev(seq_ids, torch.int32, "seq_ids"); _dev(prefix_len, torch.int32, "prefix_len")
        if tuple(vis.shape) != (batch, n_q):
            raise ValueError("vis must be [batch, n_q]")
        if seq_ids.numel() != batch or prefix_len.numel() != batch:
            raise ValueError("seq_ids and prefix_len must be [batch]")
        if out is None:
            out = torch.empty_like(q)
        self._check("sdlm_block_attn_masked_prefix", self.lib.sdlm_block_attn_masked_prefix(
            self.ctx, batch, n_q, n_k, _ptr(seq_ids), _ptr(prefix_len), _ptr(q), _ptr(k_blk), _ptr(v_blk), _ptr(vis),
            _ptr(_dev(out, torch.bfloat16, "out")), _stream_ptr(stream)))
        return out

    def verify_commit(self, draft_token: torch.Tensor, verify_token: torch.Tensor, k_blk: torch.Tensor,
                      v_blk: torch.Tensor, accepted_len: Optional[torch.Tensor] = None,
                      out_tokens: Optional[torch.Tensor] = None, seq_ids: Optional[torch.Tensor] = None, stream=None):
        batch, D = int(k_blk.shape[0]), int(k_blk.shape[1])
        _dev(draft_token, torch.int32, "draft_token"); _dev(verify_token, torch.int32, "verify_token")
        _dev(k_blk, torch.bfloat16, "k_blk"); _dev(v_blk, torch.bfloat16, "v_blk")
        if accepted_len is None:
            accepted_len = torch.empty(batch, dtype=torch.int32, device=self.device)
        if out_tokens is None:
            out_tokens = torch.empty((batch, D), dtype=torch.int32, device=self.device)
        if seq_ids is not None:
            _dev(seq_ids, torch.int32, "seq_ids")
        self._check("sdlm_verify_commit", self.lib.sdlm_verify_commit(
            self.ctx, batch, D, _ptr(seq_ids), _ptr(draft_token), _ptr(verify_token), _ptr(k_blk), _ptr(v_blk),
            _ptr(_dev(accepted_len, torch.int32, "accepted_len")), _ptr(_dev(out_tokens, torch.int32, "out_tokens")),
            _stream_ptr(stream)))
        return accepted_len, out_tokens

    def accept_commit_carry(self, tau: float, carry_len: torch.Tensor, c_max: int, token: torch.Tensor,
                            p_top1: torch.Tensor, entropy: torch.Tensor, k_rows: torch.Tensor, v_rows: torch.Tensor,
                            mode: int = CONF_LOGIT, accepted_len: Optional[torch.Tensor] = None,
                            out_tokens: Optional[torch.Tensor] = None, seq_ids: Optional[torch.Tensor] = None,
                            next_carry_len: Optional[torch.Tensor] = None, stream=None):
        """sdlm_accept_commit_carry: k_rows / v_rows are [batch, c_max + D, Hkv, d]; next_carry_len (int32
        [batch] on the device, may be carry_len itself) receives the next step's carry lengths."""
        batch, D = int(token.shape[0]), int(token.shape[1])
        _dev(carry_len, torch.int32, "carry_len"); _dev(token, torch.int32, "token")
        _dev(p_top1, torch.float32, "p_top1"); _dev(entropy, torch.float32, "entropy")
        _dev(k_rows, torch.bfloat16, "k_rows"); _dev(v_rows, torch.bfloat16, "v_rows")
        if int(k_rows.shape[1]) != c_max + D:
            raise ValueError("k_rows must hold c_max + D rows per sequence")
        if accepted_len is None:
            accepted_len = torch.empty(batch, dtype=torch.int32, device=self.device)
        if out_tokens is None:
            out_tokens = torch.empty((batch, D), dtype=torch.int32, device=self.device)
        if seq_ids is not None:
            _dev(seq_ids, torch.int32, "seq_ids")
        self._check("sdlm_accept_commit_carry", self.lib.sdlm_accept_commit_carry(
            self.ctx, batch, D, int(c_max), _ptr(seq_ids), _ptr(carry_len), float(tau), int(mode), _ptr(token),
            _ptr(p_top1), _ptr(entropy), _ptr(k_rows), _ptr(v_rows),
            _ptr(_dev(accepted_len, torch.int32, "accepted_len")), _ptr(_dev(out_tokens, torch.int32, "out_tokens")),
            _ptr(_dev(next_carry_len, torch.int32, "next_carry_len")) if next_carry_len is not None else None,
            _stream_ptr(stream)))
        return accepted_len, out_tokens

    def linear(self, x: torch.Tensor, w: torch.Tensor, bias: Optional[torch.Tensor] = None,
               residual: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        """sdlm_linear: out = x w^T (+ bias) (+ residual); x [rows, K], w [N, K]."""
        _dev(x, torch.bfloat16, "x"); _dev(w, torch.bfloat16, "w")
        K, N = int(w.shape[1]), int(w.shape[0])
        rows = x.numel() // K
        if out is None:
            out = torch.empty((rows, N), dtype=torch.bfloat16, device=self.device)
        self._check("sdlm_linear", self.lib.sdlm_linear(self.ctx, rows, K, N, _ptr(x), _ptr(w), _ptr(bias), _ptr(residual),
                                                        _ptr(_dev(out, torch.bfloat16, "out")), _stream_ptr(stream)))
        return out

    def linear_rmsnorm(self, x: torch.Tensor, w: torch.Tensor, norm_weight: torch.Tensor, eps: float,
                       bias: Optional[torch.Tensor] = None, residual: Optional[torch.Tensor] = None,
                       out: Optional[torch.Tensor] = None, norm_out: Optional[torch.Tensor] = None, stream=None):
        """sdlm_linear_rmsnorm: out = x w^T (+ bias) (+ residual) and norm_out = RMSNorm(out) * norm_weight."""
        _dev(x, torch.bfloat16, "x"); _dev(w, torch.bfloat16, "w"); _dev(norm_weight, torch.bfloat16, "norm_weight")
        K, N = int(w.shape[1]), int(w.shape[0])
        rows = x.numel() // K
        if out is None:
            out = torch.empty((rows, N), dtype=torch.bfloat16, device=self.device)
        if norm_out is None:
            norm_out = torch.empty((rows, N), dtype=torch.bfloat16, device=self.device)
        self._check("sdlm_linear_rmsnorm", self.lib.sdlm_linear_rmsnorm(
            self.ctx, rows, K, N, _ptr(x), _ptr(w), _ptr(bias), _ptr(residual), _ptr(_dev(out, torch.bfloat16, "out")),
            _ptr(norm_weight), float(eps), _ptr(_dev(norm_out, torch.bfloat16, "norm_out")), _stream_ptr(stream)))
        return out, norm_out

    def linear3(self, x: torch.Tensor, w: torch.Tensor, bias: Optional[torch.Tensor], out1: torch.Tensor,
                out2: torch.Tensor, out3: torch.Tensor, stream=None) -> None:
        """sdlm_linear3: x w^T (+ bias) with the output columns dealt to three dense tensors."""
        _dev(x, torch.bfloat16, "x"); _dev(w, torch.bfloat16, "w")
        K = int(w.shape[1])
        rows = x.numel() // K
        n = [t.numel() // rows for t in (out1, out2, out3)]
        if sum(n) != int(w.shape[0]):
            raise ValueError("the three outputs must take all of w's rows")
        self._check("sdlm_linear3", self.lib.sdlm_linear3(self.ctx, rows, K, n[0], n[1], n[2], _ptr(x), _ptr(w), _ptr(bias),
                                                          _ptr(_dev(out1, torch.bfloat16, "out1")),
                                                          _ptr(_dev(out2, torch.bfloat16, "out2")),
                                                          _ptr(_dev(out3, torch.bfloat16, "out3")), _stream_ptr(stream)))

    def linear3_rope(self, x: torch.Tensor, w: torch.Tensor, bias: Optional[torch.Tensor], q: torch.Tensor, k: torch.Tensor,
                     v: torch.Tensor, theta: float, seq_ids: Optional[torch.Tensor] = None, stream=None) -> None:
        """sdlm_linear3_rope: q [batch, D, n_heads, d], k and v [batch, D, n_heads2, d] from x [batch * D, K] and the
        stacked weight; q and k come out rotated."""
        _dev(x, torch.bfloat16, "x"); _dev(w, torch.bfloat16, "w")
        batch, D, K = int(q.shape[0]), int(q.shape[1]), int(w.shape[1])
        if x.numel() != batch * D * K or k.shape != v.shape or tuple(k.shape[:2]) != (batch, D):
            raise ValueError("x must be [batch * D, K]; k and v [batch, D, n_heads2, d]")
        if (int(q.shape[2]) + 2 * int(k.shape[2])) * int(q.shape[3]) != int(w.shape[0]):
            raise ValueError("the three outputs must take all of w's rows")
        self._check("sdlm_linear3_rope", self.lib.sdlm_linear3_rope(
            self.ctx, batch, D, _ptr(seq_ids), K, int(q.shape[2]), int(k.shape[2]), _ptr(x), _ptr(w), _ptr(bias),
            _ptr(_dev(q, torch.bfloat16, "q")), _ptr(_dev(k, torch.bfloat16, "k")), _ptr(_dev(v, torch.bfloat16, "v")),
            float(theta), _stream_ptr(stream)))

    def linear_swiglu(self, x: torch.Tensor, w_interleaved: torch.Tensor, out: Optional[torch.Tensor] = None,
                      stream=None) -> torch.Tensor:
        """sdlm_linear_swiglu: w_interleaved [2I, K] = gate_0, up_0, gate_1, up_1, ...; out [rows, I]."""
        _dev(x, torch.bfloat16, "x"); _dev(w_interleaved, torch.bfloat16, "w_interleaved")
        K, I = int(w_interleaved.shape[1]), int(w_interleaved.shape[0]) // 2
        rows = x.numel() // K
        if out is None:
            out = torch.empty((rows, I), dtype=torch.bfloat16, device=self.device)
        self._check("sdlm_linear_swiglu", self.lib.sdlm_linear_swiglu(self.ctx, rows, K, I, _ptr(x), _ptr(w_interleaved),
                                                                      _ptr(_dev(out, torch.bfloat16, "out")),
                                                                      _stream_ptr(stream)))
        return out

    def rmsnorm(self, x: torch.Tensor, weight: torch.Tensor, eps: float, out: Optional[torch.Tensor] = None,
                stream=None) -> torch.Tensor:
        _dev(x, torch.bfloat16, "x"); _dev(weight, torch.bfloat16, "weight")
        H = int(weight.numel())
        if out is None:
            out = torch.empty_like(x)
        self._check("sdlm_rmsnorm", self.lib.sdlm_rmsnorm(self.ctx, x.numel() // H, H, _ptr(x), _ptr(weight), float(eps),
                                                          _ptr(_dev(out, torch.bfloat16, "out")), _stream_ptr(stream)))
        return out

    def rope_block(self, x: torch.Tensor, theta: float, seq_ids: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        """sdlm_rope_block, in place: x [batch, D, n_heads, head_dim]."""
        _dev(x, torch.bfloat16, "x")
        batch, D, n_heads = int(x.shape[0]), int(x.shape[1]), int(x.shape[2])
        self._check("sdlm_rope_block", self.lib.sdlm_rope_block(self.ctx, batch, D, _ptr(seq_ids), n_heads, _ptr(x),
                                                                float(theta), _stream_ptr(stream)))
        return x

    def rope_block2(self, x: torch.Tensor, x2: torch.Tensor, theta: float, seq_ids: Optional[torch.Tensor] = None,
                    stream=None) -> None:
        """sdlm_rope_block2, in place: x [batch, D, n_heads, d] and x2 [batch, D, n_heads2, d] in one launch."""
        _dev(x, torch.bfloat16, "x"); _dev(x2, torch.bfloat16, "x2")
        batch, D = int(x.shape[0]), int(x.shape[1])
        self._check("sdlm_rope_block2", self.lib.sdlm_rope_block2(self.ctx, batch, D, _ptr(seq_ids), int(x.shape[2]), _ptr(x),
                                                                  int(x2.shape[2]), _ptr(x2), float(theta),
                                                                  _stream_ptr(stream)))

    def swiglu(self, gate_up: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        _dev(gate_up, torch.bfloat16, "gate_up")
        I = int(gate_up.shape[-1]) // 2
        rows = gate_up.numel() // (2 * I)
        if out is None:
            out = torch.empty((rows, I), dtype=torch.bfloat16, device=self.device)
        self._check("sdlm_swiglu", self.lib.sdlm_swiglu(self.ctx, rows, I, _ptr(gate_up),
                                                        _ptr(_dev(out, torch.bfloat16, "out")), _stream_ptr(stream)))
        return out

    def lmhead_confidence_static(self, hidden: torch.Tensor, w_lm: torch.Tensor, token: torch.Tensor,
                                 p_top1: torch.Tensor, entropy: torch.Tensor, max_logit: Optional[torch.Tensor] = None,
                                 lse: Optional[torch.Tensor] = None, stream=None) -> None:
        """sdlm_lmhead_confidence_static: the caller passes every output; nothing is allocated here."""
        _dev(hidden, torch.bfloat16, "hidden"); _dev(w_lm, torch.bfloat16, "w_lm")
        rows = hidden.numel() // self.cfg.hidden
        self._check("sdlm_lmhead_confidence_static", self.lib.sdlm_lmhead_confidence_static(
            self.ctx, rows, _ptr(hidden), _ptr(w_lm), _ptr(_dev(token, torch.int32, "token")),
            _ptr(_dev(p_top1, torch.float32, "p_top1")), _ptr(_dev(entropy, torch.float32, "entropy")),
            _ptr(max_logit), _ptr(lse), _stream_ptr(stream)))

    def lmhead_confidence(self, hidden: torch.Tensor, w_lm: torch.Tensor, token: Optional[torch.Tensor] = None,
                          p_top1: Optional[torch.Tensor] = None, entropy: Optional[torch.Tensor] = None,
                          max_logit: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None, stream=None):
        _dev(hidden, torch.bfloat16, "hidden"); _dev(w_lm, torch.bfloat16, "w_lm")
        rows = hidden.numel() // self.cfg.hidden
        shape = tuple(hidden.shape[:-1])
        if token is None:
            token = torch.empty(shape, dtype=torch.int32, device=self.device)
        if p_top1 is None:
            p_top1 = torch.empty(shape, dtype=torch.float32, device=self.device)
        if entropy is None:
            entropy = torch.empty(shape, dtype=torch.float32, device=self.device)
        self._check("sdlm_lmhead_confidence", self.lib.sdlm_lmhead_confidence(
            self.ctx, rows, _ptr(hidden), _ptr(w_lm), _ptr(_dev(token, torch.int32, "token")),
            _ptr(_dev(p_top1, torch.float32, "p_top1")), _ptr(_dev(entropy, torch.float32, "entropy")),
            _ptr(max_logit), _ptr(lse), _stream_ptr(stream)))
        return token, p_top1, entropy

    def accept_commit(self, tau: float, token: torch.Tensor, p_top1: torch.Tensor, entropy: torch.Tensor,
                      k_blk: torch.Tensor, v_blk: torch.Tensor, mode: int = CONF_LOGIT,
                      accepted_len: Optional[torch.Tensor] = None, out_tokens: Optional[torch.Tensor] = None,
                      seq_ids: Optional[torch.Tensor] = None, stream=None):
        batch, D = int(k_blk.shape[0]), int(k_blk.shape[1])
        _dev(token, torch.int32, "token"); _dev(p_top1, torch.float32, "p_top1"); _dev(entropy, torch.float32, "entropy")
        _dev(k_blk, torch.bfloat16, "k_blk"); _dev(v_blk, torch.bfloat16, "v_blk")
        if accepted_len is None:
            accepted_len = torch.empty(batch, dtype=torch.int32, device=self.device)
        if out_tokens is None:
            out_tokens = torch.empty((batch, D), dtype=torch.int32, device=self.device)
        if seq_ids is not None:
            _dev(seq_ids, torch.int32, "seq_ids")
        self._check("sdlm_accept_commit", self.lib.sdlm_accept_commit(
            self.ctx, batch, D, _ptr(seq_ids), float(tau), int(mode), _ptr(token), _ptr(p_top1), _ptr(entropy),
            _ptr(k_blk), _ptr(v_blk), _ptr(_dev(accepted_len, torch.int32, "accepted_len")),
            _ptr(_dev(out_tokens, torch.int32, "out_tokens")), _stream_ptr(stream)))
        return accepted_len, out_tokens

    def device_status(self, clear: bool = False, stream=None) -> np.ndarray:
        out = np.zeros(4, dtype=np.int32)
        self._check("sdlm_device_status", self.lib.sdlm_device_status(self.ctx, out.ctypes.data, int(clear),
                                                                      _stream_ptr(stream)))
        return out

    def decode_step(self, tau: float, q: torch.Tensor, k_blk: torch.Tensor, v_blk: torch.Tensor, hidden: torch.Tensor,
                    w_lm: torch.Tensor, attn_out: torch.Tensor, token: torch.Tensor, p_top1: torch.Tensor,
                    entropy: torch.Tensor, accepted_len: torch.Tensor, out_tokens: torch.Tensor,
                    seq_ids: Optional[torch.Tensor] = None, mode: int = CONF_LOGIT, stream=None) -> None:
        """Whole step on device tensors: attention, LM-head statistics, accept + commit."""
        batch, D = int(q.shape[0]), int(q.shape[1])
        for t, n in ((q, "q"), (k_blk, "k_blk"), (v_blk, "v_blk"), (hidden, "hidden"), (w_lm, "w_lm"), (attn_out, "attn_out")):
            _dev(t, torch.bfloat16, n)
        _dev(token, torch.int32, "token"); _dev(p_top1, torch.float32, "p_top1"); _dev(entropy, torch.float32, "entropy")
        _dev(accepted_len, torch.int32, "accepted_len"); _dev(out_tokens, torch.int32, "out_tokens")
        self._check("sdlm_decode_step", self.lib.sdlm_decode_step(
            self.ctx, batch, D, _ptr(seq_ids), float(tau), int(mode), _ptr(q), _ptr(k_blk), _ptr(v_blk), _ptr(hidden),
            _ptr(w_lm), _ptr(attn_out), _ptr(token), _ptr(p_top1), _ptr(entropy), _ptr(accepted_len),
            _ptr(out_tokens), _stream_ptr(stream)))

    def decode_step_host(self, tau: float, q: torch.Tensor, k_blk: torch.Tensor, v_blk: torch.Tensor,
                         hidden: torch.Tensor, w_lm: torch.Tensor, attn_out: Optional[torch.Tensor] = None,
                         token: Optional[torch.Tensor] = None, p_top1: Optional[torch.Tensor] = None,
                         entropy: Optional[torch.Tensor] = None, accepted_len: Optional[torch.Tensor] = None,
                         out_tokens: Optional[torch.Tensor] = None, seq_ids: Optional[torch.Tensor] = None,
                         mode: int = CONF_LOGIT, stream=None) -> None:
        """Whole step with HOST block inputs / outputs (w_lm stays on the device)."""
        batch, D = int(q.shape[0]), int(q.shape[1])
        for t, n in ((q, "q"), (k_blk, "k_blk"), (v_blk, "v_blk"), (hidden, "hidden")):
            _host(t, torch.bfloat16, n)
        _dev(w_lm, torch.bfloat16, "w_lm")
        self._check("sdlm_decode_step_host", self.lib.sdlm_decode_step_host(
            self.ctx, batch, D, _ptr(seq_ids), float(tau), int(mode), _ptr(q), _ptr(k_blk), _ptr(v_blk), _ptr(hidden),
            _ptr(w_lm), _ptr(attn_out), _ptr(token), _ptr(p_top1), _ptr(entropy), _ptr(accepted_len),
            _ptr(out_tokens), _stream_ptr(stream)))

    def selftest_bounded_wait(self, stream=None) -> None:
        self._check("sdlm_selftest_bounded_wait", self.lib.sdlm_selftest_bounded_wait(self.ctx, _stream_ptr(stream)))

    def set_option(self, opt: int, value: int) -> None:
        self._check("sdlm_set_option", self.lib.sdlm_set_option(self.ctx, opt, value))

    def launch_count(self) -> int:
        return int(self.lib.sdlm_launch_count(self.ctx))
