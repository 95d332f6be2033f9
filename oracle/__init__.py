"""TEST INFRASTRUCTURE -- the fp64 CPU oracle of the cloud-side verification step.

Thin ctypes access to ``flexspec_oracle.c`` (Algorithm 2, Step 2; Section IV-C).
Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA path never does, and nothing here imports the CUDA path.

All arrays are numpy; bf16 tensors travel as ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "flexspec_oracle.c")
_HDR = os.path.join(_HERE, "flexspec_oracle.h")
# FLEXSPEC_ORACLE_SANITIZE=1: a separate build with AddressSanitizer + UndefinedBehaviorSanitizer (the
# process must then run with libasan preloaded; tests/test_oracle_sanitized.py does that in a child)
_SANITIZE = os.environ.get("FLEXSPEC_ORACLE_SANITIZE", "") == "1"
_LIB = os.path.join(_HERE, "libflexspec_oracle_san.so" if _SANITIZE else "libflexspec_oracle.so")

GREEDY = 1
SAMPLE = 0


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP, no fast-math)."""
    stale = (not os.path.exists(_LIB)
             or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_HDR)))
    if force or stale:
        opt = ["-O1", "-g", "-fsanitize=address,undefined", "-fno-omit-frame-pointer"] if _SANITIZE else ["-O2"]
        cmd = ["gcc"] + opt + ["-std=c11", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra",
                                "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(_LIB)
        vp, i32, f64 = C.c_void_p, C.c_int32, C.c_double
        L.fso_bf16_to_f64.restype = f64
        L.fso_bf16_to_f64.argtypes = [C.c_uint16]
        L.fso_f64_to_bf16.restype = C.c_uint16
        L.fso_f64_to_bf16.argtypes = [f64]
        L.fso_philox4x32_10.restype = None
        L.fso_philox4x32_10.argtypes = [vp, vp, vp]
        L.fso_uniform.restype = f64
        L.fso_uniform.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32]
        L.fso_attention.restype = None
        L.fso_attention.argtypes = [vp, vp, vp, i32, vp, vp, i32, i32, i32, i32, i32, vp, i32, vp, vp]
        L.fso_lm_head.restype = None
        L.fso_lm_head.argtypes = [vp, vp, i32, i32, i32, vp, i32, vp]
        L.fso_softmax.restype = None
        L.fso_softmax.argtypes = [vp, i32, f64, vp, vp]
        L.fso_accept.restype = None
        L.fso_accept.argtypes = [i32, vp, vp, vp, vp, vp, i32, i32, f64, vp, i32, f64, vp, vp, i32,
                                 vp, vp, vp, vp, vp, vp, vp, vp, vp]
        L.fso_emission.restype = f64
        L.fso_emission.argtypes = [vp, vp, i32, f64, i32, f64, vp, vp, vp]
        L.fso_topk.restype = None
        L.fso_topk.argtypes = [vp, i32, i32]
        L.fso_kv_release.restype = None
        L.fso_kv_release.argtypes = [vp, i32, vp, vp, i32, i32, vp, vp]
        L.fso_nucleus.restype = None
        L.fso_nucleus.argtypes = [vp, i32, f64, vp]
        L.fso_kv_append.restype = None
        L.fso_kv_append.argtypes = [vp, vp, i32, vp, vp, i32, i32, i32, i32, vp, vp]
        L.fso_kv_rollback.restype = None
        L.fso_kv_rollback.argtypes = [vp, vp, vp, i32, vp]
        L.fso_num_threads.restype = i32
        _lib = L
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _c(a, dtype):
    if a is None:
        return None
    return np.ascontiguousarray(a, dtype=dtype)


def num_threads() -> int:
    return int(lib().fso_num_threads())


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact decode of bf16 bit patterns (uint16) to float64."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f64_to_bf16(x: np.ndarray) -> np.ndarray:
    L = lib()
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty(x.shape, dtype=np.uint16)
    xf, of = x.reshape(-1), out.reshape(-1)
    for i in range(xf.size):
        of[i] = L.fso_f64_to_bf16(float(xf[i]))
    return out


def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().fso_philox4x32_10(_p(c), _p(k), _p(out))
    return out


def uniform(seed: int, index: int, stream: int) -> float:
    return float(lib().fso_uniform(C.c_uint64(seed), index, stream))


def attention(hidden, kv_pages, page_table, kv_len, draft_len, n_q_heads, n_kv_heads,
              head_dim, page_size=16, seq_sel=None):
    """Returns (attn_f64 [M,d], attn_bf16 bits [M,d]); rows of unselected sequences are 0."""
    hidden = _c(hidden, np.uint16)
    kv_pages = _c(kv_pages, np.uint16)
    page_table = _c(page_table, np.int32)
    kv_len = _c(kv_len, np.int32)
    draft_len = _c(draft_len, np.int32)
    batch = int(draft_len.shape[0])
    m = int(draft_len.sum()) + batch
    d = n_q_heads * head_dim
    assert hidden.size == m * d, (hidden.shape, m, d)
    sel = _c(seq_sel, np.int32)
    out64 = np.zeros((m, d), dtype=np.float64)
    out16 = np.zeros((m, d), dtype=np.uint16)
    lib().fso_attention(_p(hidden), _p(kv_pages), _p(page_table), int(page_table.shape[1]),
                        _p(kv_len), _p(draft_len), batch, n_q_heads, n_kv_heads, head_dim,
                        page_size, _p(sel), 0 if sel is None else int(sel.size),
                        _p(out64), _p(out16))
    return out64, out16


def lm_head(x_bf16, w_bf16, row_sel=None):
    """logits fp64 [M,V] = x [M,d] . w[V,d]^T; unselected rows are 0."""
    x = _c(x_bf16, np.uint16)
    w = _c(w_bf16, np.uint16)
    m, d = x.shape
    v = w.shape[0]
    assert w.shape[1] == d
    sel = _c(row_sel, np.int32)
    out = np.zeros((m, v), dtype=np.float64)
    lib().fso_lm_head(_p(x), _p(w), m, d, v, _p(sel), 0 if sel is None else int(sel.size), _p(out))
    return out


def softmax(z, temperature=1.0, mask=None):
    z = _c(z, np.float64)
    mask = _c(mask, np.uint32)
    out = np.empty_like(z)
    lib().fso_softmax(_p(z), int(z.size), float(temperature), _p(mask), _p(out))
    return out


def nucleus(prob, top_p):
    """Top-p filtered and renormalised copy of a distribution; returns (prob', margin)."""
    p = np.array(prob, dtype=np.float64, copy=True)
    m = np.zeros(1, dtype=np.float64)
    lib().fso_nucleus(_p(p), int(p.size), float(top_p), _p(m))
    return p, float(m[0])


def topk(prob, top_k):
    """Top-k filtered and renormalised copy of a distribution (ties with the k-th token are all kept)."""
    p = np.array(prob, dtype=np.float64, copy=True)
    lib().fso_topk(_p(p), int(p.size), int(top_k))
    return p


def emission(target_row, draft_row=None, temperature=1.0, top_p=1.0, mask=None, top_k=0):
    """Unnormalised weights r[v] of the emitted token and their sum Z for one target row: the residual
    max(0, p - q) when a draft row is given (first rejection), p itself otherwise (bonus row)."""
    zt = _c(target_row, np.float64)
    zd = _c(draft_row, np.float32)
    mask = _c(mask, np.uint32)
    r = np.empty(zt.shape[0], dtype=np.float64)
    z = lib().fso_emission(_p(zt), _p(zd), int(zt.shape[0]), float(temperature), int(top_k), float(top_p), _p(mask), _p(r), None)
    return r, float(z)


def accept(mode, target_logits, draft_logits, draft_tokens, draft_len, seeds, temperature=1.0,
           vocab_mask=None, seq_sel=None, top_p=1.0, top_k=0, temperatures=None):
    """Acceptance loop + emitted token.  Returns a dict of numpy arrays.  `temperatures`: one value per
    sequence (overrides `temperature`); top_k / top_p filter the target distribution."""
    zt = _c(target_logits, np.float64)
    zd = _c(draft_logits, np.float32)
    x = _c(draft_tokens, np.int32)
    k = _c(draft_len, np.int32)
    seeds = _c(seeds, np.uint64)
    mask = _c(vocab_mask, np.uint32)
    sel = _c(seq_sel, np.int32)
    batch = int(k.shape[0])
    vocab = int(zt.shape[-1])
    s = int(k.sum())
    assert zt.size == (s + batch) * vocab
    if mode == SAMPLE:
        assert zd is not None and zd.size == s * vocab
    if x is None or x.size == 0:
        x = np.zeros(1, dtype=np.int32)
    res = {
        "accepted_len": np.full(batch, -1, dtype=np.int32),
        "next_token": np.full(batch, -1, dtype=np.int32),
        "p_tok": np.zeros(s, dtype=np.float64),
        "q_tok": np.zeros(s, dtype=np.float64),
        "u": np.zeros(s, dtype=np.float64),
        "acc_margin": np.full(s, np.inf, dtype=np.float64),
        "cdf_margin": np.full(batch, np.inf, dtype=np.float64),
        "resid_mass": np.zeros(batch, dtype=np.float64),
        "topp_margin": np.full(s + batch, np.inf, dtype=np.float64),
    }
    temps = _c(temperatures, np.float64)
    assert temps is None or temps.size == batch
    lib().fso_accept(int(mode), _p(zt), _p(zd), _p(x), _p(k), _p(seeds), batch, vocab,
                     float(temperature), _p(temps), int(top_k), float(top_p), _p(mask), _p(sel), 0 if sel is None else int(sel.size),
                     _p(res["accepted_len"]), _p(res["next_token"]), _p(res["p_tok"]),
                     _p(res["q_tok"]), _p(res["u"]), _p(res["acc_margin"]),
                     _p(res["cdf_margin"]), _p(res["resid_mass"]), _p(res["topp_margin"]))
    return res


def kv_append(kv_pages, page_table, kv_len, draft_len, new_k, new_v, n_kv_heads, head_dim, page_size=16):
    """Returns a copy of the pool (uint16 bit patterns) with the window rows written (Section IV-C)."""
    pool = np.array(kv_pages, dtype=np.uint16, copy=True)
    page_table = _c(page_table, np.int32)
    kv_len = _c(kv_len, np.int32)
    draft_len = _c(draft_len, np.int32)
    nk, nv = _c(new_k, np.uint16), _c(new_v, np.uint16)
    lib().fso_kv_append(_p(pool), _p(page_table), int(page_table.shape[1]), _p(kv_len), _p(draft_len),
                        int(draft_len.shape[0]), n_kv_heads, head_dim, page_size, _p(nk), _p(nv))
    return pool


def kv_rollback(kv_len, draft_len, accepted_len):
    kv_len, draft_len, accepted_len = _c(kv_len, np.int32), _c(draft_len, np.int32), _c(accepted_len, np.int32)
    out = np.empty_like(kv_len)
    lib().fso_kv_rollback(_p(kv_len), _p(draft_len), _p(accepted_len), int(kv_len.shape[0]), _p(out))
    return out


def kv_release(page_table, kv_len_prev, kv_len_next, page_size=16):
    """Returns (page table with the released entries set to -1, released page ids in order)."""
    pt = np.array(page_table, dtype=np.int32, copy=True)
    prev, nxt = _c(kv_len_prev, np.int32), _c(kv_len_next, np.int32)
    free = np.full(pt.size, -1, dtype=np.int32)
    cnt = np.zeros(1, dtype=np.int32)
    lib().fso_kv_release(_p(pt), int(pt.shape[1]), _p(prev), _p(nxt), int(pt.shape[0]), page_size, _p(free), _p(cnt))
    return pt, free[:int(cnt[0])]


def verify(mode, hidden, kv_pages, page_table, kv_len, draft_len, lm_head_w, draft_tokens,
           draft_logits, seeds, n_q_heads, n_kv_heads, head_dim, page_size=16, temperature=1.0,
           vocab_mask=None, seq_sel=None, top_p=1.0, top_k=0, temperatures=None):
    """The whole step in the order of Algorithm 2, Step 2: attention over the
    restored KV session -> bf16 -> LM head -> acceptance loop -> emitted token."""
    draft_len = _c(draft_len, np.int32)
    attn64, attn16 = attention(hidden, kv_pages, page_table, kv_len, draft_len, n_q_heads,
                               n_kv_heads, head_dim, page_size, seq_sel)
    row_sel = None
    if seq_sel is not None:
        row0 = np.concatenate([[0], np.cumsum(draft_len + 1)])
        row_sel = np.concatenate([np.arange(row0[b], row0[b + 1]) for b in seq_sel]).astype(np.int32)
    logits = lm_head(attn16, lm_head_w, row_sel)
    res = accept(mode, logits, draft_logits, draft_tokens, draft_len, seeds, temperature,
                 vocab_mask, seq_sel, top_p=top_p, top_k=top_k, temperatures=temperatures)
    res["attn_f64"] = attn64
    res["attn_bf16"] = attn16
    res["logits"] = logits
    return res
