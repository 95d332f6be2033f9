"""Thin Python binding of the C ABI in include/flexspec.h (argument marshalling only).

Every step of the verification step runs in the CUDA library; torch is used for device
memory and streams.  Importing this module loads ``lib/libflexspec.so`` and raises if it
is missing -- there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

from . import build as _build

MODE_SAMPLE = 0
MODE_GREEDY = 1
FLAG_DEBUG = 1

OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_OOM, ERR_CUDA = -1, -2, -3, -4
ERR_TIMEOUT, ERR_BAD_PAGE, ERR_BAD_TOKEN, ERR_NO_DEVICE = -5, -6, -7, -8

EXPORTS = [
    "flexspec_create", "flexspec_verify", "flexspec_verify_host", "flexspec_attention",
    "flexspec_lm_head", "flexspec_sample", "flexspec_sample_static", "flexspec_kv_append",
    "flexspec_kv_rollback", "flexspec_kv_release", "flexspec_set_top_p", "flexspec_set_sampling", "flexspec_get_debug", "flexspec_status",
    "flexspec_selftest_wait_timeout", "flexspec_set_profiling", "flexspec_get_stage_ms", "flexspec_last_launches",
    "flexspec_destroy", "flexspec_strerror", "flexspec_version",
]


class Config(C.Structure):
    _fields_ = [("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("vocab", C.c_int32), ("page_size", C.c_int32), ("max_batch", C.c_int32),
                ("k_max", C.c_int32), ("max_kv_len", C.c_int32), ("mode", C.c_int32),
                ("device", C.c_int32), ("flags", C.c_uint32)]


class KV(C.Structure):
    _fields_ = [("kv_pages", C.c_void_p), ("num_pages", C.c_int32), ("page_table", C.c_void_p),
                ("max_pages_per_seq", C.c_int32), ("kv_len", C.c_void_p), ("kv_len_host", C.c_void_p)]


class Debug(C.Structure):
    _fields_ = [("attn_out", C.c_void_p), ("logits", C.c_void_p), ("p_tok", C.c_void_p),
                ("q_tok", C.c_void_p), ("u_acc", C.c_void_p), ("status", C.c_void_p), ("topp", C.c_void_p)]


def _load() -> C.CDLL:
    path = _build.LIB_PATH
    if not os.path.exists(path):
        raise ImportError(
            f"{path} is missing: build it with `python -m paper_2601_00644_b200.build` "
            "(needs nvcc); the verification step has no other implementation")
    lib = C.CDLL(path)
    vp, i32, f32 = C.c_void_p, C.c_int32, C.c_float
    lib.flexspec_create.argtypes = [C.POINTER(Config), vp, C.POINTER(vp)]
    lib.flexspec_verify.argtypes = [vp, C.POINTER(KV), vp, vp, vp, vp, vp, vp, i32, f32, vp, vp, vp, vp]
    lib.flexspec_verify_host.argtypes = [vp, C.POINTER(KV), vp, vp, vp, vp, vp, i32, f32, vp, vp, vp, vp]
    lib.flexspec_attention.argtypes = [vp, C.POINTER(KV), vp, vp, vp, i32, vp, vp]
    lib.flexspec_lm_head.argtypes = [vp, vp, i32, vp, vp]
    lib.flexspec_sample.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, f32, vp, vp, vp, vp]
    lib.flexspec_sample_static.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, f32, vp, vp, vp, vp]
    lib.flexspec_kv_append.argtypes = [vp, vp, i32, vp, i32, vp, vp, vp, vp, vp, vp, i32, vp]
    lib.flexspec_kv_rollback.argtypes = [vp, vp, vp, vp, i32, vp, vp]
    lib.flexspec_kv_release.argtypes = [vp, vp, i32, i32, vp, vp, i32, vp, i32, vp, vp]
    lib.flexspec_set_top_p.argtypes = [vp, f32]
    lib.flexspec_set_sampling.argtypes = [vp, f32, i32, vp]
    lib.flexspec_get_debug.argtypes = [vp, C.POINTER(Debug)]
    lib.flexspec_status.argtypes = [vp, vp]
    lib.flexspec_selftest_wait_timeout.argtypes = [vp, C.c_int64, vp]
    lib.flexspec_set_profiling.argtypes = [vp, i32]
    lib.flexspec_get_stage_ms.argtypes = [vp, vp]
    lib.flexspec_last_launches.argtypes = [vp]
    lib.flexspec_destroy.argtypes = [vp]
    lib.flexspec_strerror.argtypes = [C.c_int]
    lib.flexspec_strerror.restype = C.c_char_p
    lib.flexspec_version.restype = C.c_char_p
    for name in EXPORTS:
        if name not in ("flexspec_strerror", "flexspec_version"):
            getattr(lib, name).restype = C.c_int
    return lib


LIB = _load()


class FlexSpecError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {LIB.flexspec_strerror(code).decode()} ({code})")


def _check(code: int, where: str):
    if code != OK:
        raise FlexSpecError(code, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream_ptr(stream: Optional[torch.cuda.Stream]):
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def _dev(t, dtype, name):
    if t is None:
        return None
    if not (t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{name}: expected a contiguous CUDA tensor of {dtype}")
    return t


def _host_i32(t, name):
    if t.is_cuda or t.dtype != torch.int32 or not t.is_contiguous():
        raise TypeError(f"{name}: expected a contiguous CPU int32 tensor")
    return t


def sample_static(logits, draft_tokens, draft_logits, draft_len, draft_len_host, seeds, mode=MODE_SAMPLE,
                  temperature=1.0, vocab_mask=None, accepted_len=None, next_token=None, stream=None):
    """flexspec_sample_static: the acceptance / emitted-token stage for hosts that cannot allocate
    device memory at call time.  No handle; the library's built-in scratch array is used, so calls
    on one device must not overlap.  Outputs may be passed in (then nothing at all is allocated,
    not even by torch); otherwise two int32 tensors are created for convenience."""
    batch = int(draft_len_host.numel())
    _dev(logits, torch.float32, "logits")
    vocab = int(logits.shape[-1])
    dev = logits.device
    if accepted_len is None:
        accepted_len = torch.empty(batch, dtype=torch.int32, device=dev)
    if next_token is None:
        next_token = torch.empty(batch, dtype=torch.int32, device=dev)
    with torch.cuda.device(dev):
        _check(LIB.flexspec_sample_static(
            _ptr(logits), _ptr(_dev(draft_tokens, torch.int32, "draft_tokens")),
            _ptr(_dev(draft_logits, torch.float32, "draft_logits")), _ptr(_dev(draft_len, torch.int32, "draft_len")),
            _ptr(_host_i32(draft_len_host, "draft_len_host")), _ptr(_dev(seeds, torch.int64, "seeds")),
            batch, vocab, int(mode), float(temperature), _ptr(_dev(vocab_mask, torch.int32, "vocab_mask")),
            _ptr(_dev(accepted_len, torch.int32, "accepted_len")), _ptr(_dev(next_token, torch.int32, "next_token")),
            _stream_ptr(stream)), "flexspec_sample_static")
    return accepted_len, next_token


class Verifier:
    """Owns one flexspec handle (workspace + LM-head descriptor) on one device."""

    def __init__(self, lm_head_w: torch.Tensor, n_q_heads: int, n_kv_heads: int, head_dim: int,
                 max_batch: int, k_max: int, max_kv_len: int, mode: int = MODE_SAMPLE,
                 debug: bool = False, page_size: int = 16):
        _dev(lm_head_w, torch.bfloat16, "lm_head_w")
        self.vocab = int(lm_head_w.shape[0])
        self.d_model = int(lm_head_w.shape[1])
        self.cfg = Config(n_q_heads, n_kv_heads, head_dim, self.vocab, page_size, max_batch, k_max,
                          max_kv_len, mode, lm_head_w.device.index or 0, FLAG_DEBUG if debug else 0)
        if n_q_heads * head_dim != self.d_model:
            raise ValueError("lm_head_w must be [vocab, n_q_heads*head_dim]")
        self.device = lm_head_w.device
        self._h = C.c_void_p()
        _check(LIB.flexspec_create(C.byref(self.cfg), _ptr(lm_head_w), C.byref(self._h)), "flexspec_create")
        self._keep = None

    # ------------------------------------------------------------------ helpers
    def _kv(self, kv_pages, page_table, kv_len, kv_len_host):
        _dev(kv_pages, torch.bfloat16, "kv_pages")
        _dev(page_table, torch.int32, "page_table")
        _host_i32(kv_len_host, "kv_len_host")
        if kv_len is not None:
            _dev(kv_len, torch.int32, "kv_len")
        return KV(kv_pages.data_ptr(), int(kv_pages.shape[0]), page_table.data_ptr(),
                  int(page_table.shape[1]), None if kv_len is None else kv_len.data_ptr(),
                  kv_len_host.data_ptr())

    # ------------------------------------------------------------------ the step
    def verify(self, kv_pages, page_table, kv_len, kv_len_host, hidden, draft_tokens, draft_logits,
               draft_len, draft_len_host, seeds, temperature=1.0, vocab_mask=None,
               accepted_len=None, next_token=None, stream=None):
        batch = int(draft_len_host.numel())
        kv = self._kv(kv_pages, page_table, kv_len, kv_len_host)
        _dev(hidden, torch.bfloat16, "hidden")
        _dev(draft_tokens, torch.int32, "draft_tokens")
        _dev(draft_logits, torch.float32, "draft_logits")
        _dev(draft_len, torch.int32, "draft_len")
        _host_i32(draft_len_host, "draft_len_host")
        _dev(seeds, torch.int64, "seeds")
        _dev(vocab_mask, torch.int32, "vocab_mask")
        if accepted_len is None:
            accepted_len = torch.empty(batch, dtype=torch.int32, device=self.device)
        if next_token is None:
            next_token = torch.empty(batch, dtype=torch.int32, device=self.device)
        _check(LIB.flexspec_verify(self._h, C.byref(kv), _ptr(hidden), _ptr(draft_tokens),
                                   _ptr(draft_logits), _ptr(draft_len), _ptr(draft_len_host),
                                   _ptr(seeds), batch, float(temperature), _ptr(vocab_mask),
                                   _ptr(accepted_len), _ptr(next_token), _stream_ptr(stream)),
               "flexspec_verify")
        return accepted_len, next_token

    def verify_host(self, kv_pages, page_table, kv_len_host, hidden, draft_tokens, draft_logits,
                    draft_len, seeds, accepted_len, next_token, temperature=1.0, stream=None, vocab_mask=None):
        """Per-step inputs and outputs are HOST tensors (pinned for speed); KV stays on the device."""
        batch = int(draft_len.numel())
        kv = self._kv(kv_pages, page_table, None, kv_len_host)
        for t, name in ((hidden, "hidden"), (draft_tokens, "draft_tokens"), (draft_logits, "draft_logits"),
                        (draft_len, "draft_len"), (seeds, "seeds"), (accepted_len, "accepted_len"),
                        (next_token, "next_token"), (vocab_mask, "vocab_mask")):
            if t is not None and (t.is_cuda or not t.is_contiguous()):
                raise TypeError(f"{name}: expected a contiguous CPU tensor")
        _check(LIB.flexspec_verify_host(self._h, C.byref(kv), _ptr(hidden), _ptr(draft_tokens),
                                        _ptr(draft_logits), _ptr(draft_len), _ptr(seeds), batch,
                                        float(temperature), _ptr(vocab_mask), _ptr(accepted_len), _ptr(next_token),
                                        _stream_ptr(stream)), "flexspec_verify_host")
        return accepted_len, next_token

    # ------------------------------------------------------------------ stages
    def attention(self, kv_pages, page_table, kv_len, kv_len_host, hidden, draft_len, draft_len_host,
                  attn_out=None, stream=None):
        batch = int(draft_len_host.numel())
        kv = self._kv(kv_pages, page_table, kv_len, kv_len_host)
        _dev(hidden, torch.bfloat16, "hidden")
        if attn_out is None:
            m = int(draft_len_host.sum().item()) + batch
            attn_out = torch.empty(m, self.d_model, dtype=torch.bfloat16, device=self.device)
        _check(LIB.flexspec_attention(self._h, C.byref(kv), _ptr(hidden), _ptr(_dev(draft_len, torch.int32, "draft_len")),
                                      _ptr(_host_i32(draft_len_host, "draft_len_host")), batch,
                                      _ptr(attn_out), _stream_ptr(stream)), "flexspec_attention")
        return attn_out

    def lm_head(self, x, logits=None, stream=None):
        _dev(x, torch.bfloat16, "x")
        m = int(x.shape[0])
        if logits is None:
            logits = torch.empty(m, self.vocab, dtype=torch.float32, device=self.device)
        _check(LIB.flexspec_lm_head(self._h, _ptr(x), m, _ptr(logits), _stream_ptr(stream)), "flexspec_lm_head")
        return logits

    def sample(self, logits, draft_tokens, draft_logits, draft_len, draft_len_host, seeds,
               temperature=1.0, vocab_mask=None, stream=None):
        batch = int(draft_len_host.numel())
        _dev(logits, torch.float32, "logits")
        accepted_len = torch.empty(batch, dtype=torch.int32, device=self.device)
        next_token = torch.empty(batch, dtype=torch.int32, device=self.device)
        _check(LIB.flexspec_sample(self._h, _ptr(logits), _ptr(_dev(draft_tokens, torch.int32, "draft_tokens")),
                                   _ptr(_dev(draft_logits, torch.float32, "draft_logits")),
                                   _ptr(_dev(draft_len, torch.int32, "draft_len")),
                                   _ptr(_host_i32(draft_len_host, "draft_len_host")),
                                   _ptr(_dev(seeds, torch.int64, "seeds")), batch, float(temperature),
                                   _ptr(_dev(vocab_mask, torch.int32, "vocab_mask")),
                                   _ptr(accepted_len), _ptr(next_token), _stream_ptr(stream)), "flexspec_sample")
        return accepted_len, next_token

    # ------------------------------------------------------------------ KV session
    def kv_append(self, kv_pages, page_table, kv_len, kv_len_host, new_k, new_v, draft_len, draft_len_host, stream=None):
        """Write the K/V rows of the window positions into the pages (before verify)."""
        batch = int(draft_len_host.numel())
        _dev(kv_pages, torch.bfloat16, "kv_pages"); _dev(new_k, torch.bfloat16, "new_k"); _dev(new_v, torch.bfloat16, "new_v")
        _check(LIB.flexspec_kv_append(self._h, _ptr(kv_pages), int(kv_pages.shape[0]), _ptr(_dev(page_table, torch.int32, "page_table")),
                                      int(page_table.shape[1]), _ptr(_dev(kv_len, torch.int32, "kv_len")),
                                      _ptr(_host_i32(kv_len_host, "kv_len_host")), _ptr(new_k), _ptr(new_v),
                                      _ptr(_dev(draft_len, torch.int32, "draft_len")), _ptr(_host_i32(draft_len_host, "draft_len_host")),
                                      batch, _stream_ptr(stream)), "flexspec_kv_append")

    def kv_rollback(self, kv_len, draft_len, accepted_len, kv_len_next=None, stream=None):
        """kv_len of the next step after this step's accepted_len (device-side, no host sync)."""
        if kv_len_next is None:
            kv_len_next = torch.empty_like(kv_len)
        _check(LIB.flexspec_kv_rollback(self._h, _ptr(_dev(kv_len, torch.int32, "kv_len")), _ptr(_dev(draft_len, torch.int32, "draft_len")),
                                        _ptr(_dev(accepted_len, torch.int32, "accepted_len")), int(kv_len.numel()),
                                        _ptr(_dev(kv_len_next, torch.int32, "kv_len_next")), _stream_ptr(stream)), "flexspec_kv_rollback")
        return kv_len_next

    def kv_release(self, page_table, num_pages, kv_len_prev, kv_len_next, free_list, free_count, stream=None):
        """Push the pages past kv_len_next onto free_list (advancing free_count) and clear their table entries."""
        _check(LIB.flexspec_kv_release(self._h, _ptr(_dev(page_table, torch.int32, "page_table")), int(page_table.shape[1]),
                                       int(num_pages), _ptr(_dev(kv_len_prev, torch.int32, "kv_len_prev")),
                                       _ptr(_dev(kv_len_next, torch.int32, "kv_len_next")), int(kv_len_prev.numel()),
                                       _ptr(_dev(free_list, torch.int32, "free_list")), int(free_list.numel()),
                                       _ptr(_dev(free_count, torch.int32, "free_count")), _stream_ptr(stream)),
               "flexspec_kv_release")

    # ------------------------------------------------------------------ introspection
    def _view(self, ptr, shape, dtype):
        """A copy of workspace memory as a torch tensor (via the CUDA array interface)."""
        typestr = {torch.bfloat16: "<i2", torch.float32: "<f4", torch.float64: "<f8", torch.int32: "<i4"}[dtype]
        n = 1
        for s in shape:
            n *= s
        if n == 0 or not ptr:
            return torch.empty(shape, dtype=dtype, device=self.device)

        class _Raw:
            pass
        raw = _Raw()
        raw.__cuda_array_interface__ = {"shape": tuple(shape), "typestr": typestr, "data": (int(ptr), False),
                                        "version": 2}
        t = torch.as_tensor(raw, device=self.device)
        if dtype == torch.bfloat16:
            t = t.view(torch.bfloat16)
        return t.clone()

    def debug(self, m_rows: int, s_rows: int):
        """Copies of the workspace intermediates of the last call (synchronises first)."""
        torch.cuda.synchronize(self.device)
        d = Debug()
        _check(LIB.flexspec_get_debug(self._h, C.byref(d)), "flexspec_get_debug")
        return {
            "attn_out": self._view(d.attn_out, (m_rows, self.d_model), torch.bfloat16),
            "logits": self._view(d.logits, (m_rows, self.vocab), torch.float32),
            "p_tok": self._view(d.p_tok, (s_rows,), torch.float64),
            "q_tok": self._view(d.q_tok, (s_rows,), torch.float64),
            "u": self._view(d.u_acc, (s_rows,), torch.float32),
            "topp": self._view(d.topp, (m_rows, 2), torch.float64),
        }

    def set_top_p(self, top_p: float):
        """Nucleus sampling of the target (1.0 = off) for the following calls."""
        _check(LIB.flexspec_set_top_p(self._h, float(top_p)), "flexspec_set_top_p")

    def set_sampling(self, top_p: float = 1.0, top_k: int = 0, temperatures: Optional[torch.Tensor] = None):
        """top-p / top-k filters of the target and per-sequence temperatures (a CUDA fp32 tensor [batch],
        kept alive here because the library only borrows it) for the following calls."""
        _dev(temperatures, torch.float32, "temperatures")
        self._temps = temperatures
        _check(LIB.flexspec_set_sampling(self._h, float(top_p), int(top_k), _ptr(temperatures)), "flexspec_set_sampling")

    def status(self):
        st = (C.c_int32 * 4)()
        code = LIB.flexspec_status(self._h, st)
        return code, list(st)

    def selftest_wait_timeout(self, limit_ns: int, stream=None):
        """Launch the diagnostic kernel whose bounded wait runs out after limit_ns (see the header)."""
        _check(LIB.flexspec_selftest_wait_timeout(self._h, int(limit_ns), _stream_ptr(stream)),
               "flexspec_selftest_wait_timeout")

    def set_profiling(self, on: bool):
        _check(LIB.flexspec_set_profiling(self._h, 1 if on else 0), "flexspec_set_profiling")

    def stage_ms(self):
        ms = (C.c_float * 6)()
        _check(LIB.flexspec_get_stage_ms(self._h, ms), "flexspec_get_stage_ms")
        return list(ms)

    def last_launches(self) -> int:
        return int(LIB.flexspec_last_launches(self._h))

    def close(self):
        if self._h:
            LIB.flexspec_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
