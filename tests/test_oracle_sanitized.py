"""The oracle under AddressSanitizer + UndefinedBehaviorSanitizer: every exported function is driven
over small ragged cases (empty drafts, partial pages, masks, filters, every mode) in a child process
with the sanitizer runtime preloaded; any out-of-bounds access, use of uninitialised stack, signed
overflow or misaligned access ends the child with a report."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

DRIVER = r'''
import numpy as np
import oracle
rng = np.random.RandomState(11)
def bf16(a):
    return (np.asarray(a, np.float32).view(np.uint32) >> 16).astype(np.uint16)
# attention + LM head over a ragged, paged batch (k = 0, partial last pages, permuted pages)
H, HKV, DH, V, B = 4, 2, 64, 97, 4
k = np.array([0, 3, 1, 5], np.int32)
ctx = np.array([0, 17, 31, 40], np.int32)
kv_len = ctx + k + 1
pages = (kv_len + 15) // 16
pt = np.full((B, int(pages.max()) + 1), -1, np.int32)
perm = rng.permutation(int(pages.sum()) + 2).astype(np.int32)
c = 0
for b in range(B):
    pt[b, :pages[b]] = perm[c:c + pages[b]]; c += pages[b]
M, S = int(k.sum()) + B, int(k.sum())
hidden = bf16(rng.standard_normal((M, H * DH)))
pool = bf16(rng.standard_normal((len(perm), 2, HKV, 16, DH)))
w = bf16(rng.standard_normal((V, H * DH)) * 0.1)
a64, a16 = oracle.attention(hidden, pool, pt, kv_len, k, H, HKV, DH)
a64s, _ = oracle.attention(hidden, pool, pt, kv_len, k, H, HKV, DH, seq_sel=[1, 3])
logits = oracle.lm_head(a16, w)
oracle.lm_head(a16, w, row_sel=np.array([0, M - 1], np.int32))
zd = (rng.standard_normal((S, V))).astype(np.float32)
toks = rng.randint(0, V, S).astype(np.int32)
seeds = rng.randint(0, 2 ** 62, B).astype(np.uint64)
mask = np.full((B, (V + 31) // 32), 0xFFFFFFFF, np.uint32); mask[1] = 0x55555555
for mode in (0, 1):
    for kw in (dict(), dict(vocab_mask=mask), dict(top_p=0.8), dict(top_k=5), dict(top_k=7, top_p=0.6),
               dict(temperatures=np.array([0.5, 1.0, 2.0, 0.7])), dict(seq_sel=[0, 2])):
        if mode == 1 and ("top_p" in kw or "top_k" in kw or "temperatures" in kw):
            continue
        r = oracle.accept(mode, logits, zd, toks, k, seeds, 0.9, **kw)
        assert ((r["accepted_len"] <= k) | (r["accepted_len"] < 0)).all()
res = oracle.verify(0, hidden, pool, pt, kv_len, k, w, toks, zd, seeds, H, HKV, DH, top_p=0.9, top_k=20)
p = rng.dirichlet(np.ones(V))
oracle.nucleus(p, 0.5); oracle.nucleus(p, 1.0); oracle.topk(p, 1); oracle.topk(p, V + 3)
oracle.emission(logits[0], zd[0] if S else None, 0.8, 0.9, mask[0], top_k=9); oracle.emission(logits[0], None)
oracle.softmax(logits[0], 0.7, mask[1])
oracle.philox4x32_10([1, 2, 3, 4], [5, 6]); oracle.uniform(12345678901234567, 3, 1)
oracle.bf16_to_f64(hidden[:3]); oracle.f64_to_bf16(np.array([1.0, -2.5, 3e38, 1e-40, np.inf]))
nk, nv = bf16(rng.standard_normal((M, HKV, DH))), bf16(rng.standard_normal((M, HKV, DH)))
oracle.kv_append(pool, pt, kv_len, k, nk, nv, HKV, DH)
nxt = oracle.kv_rollback(kv_len, k, np.minimum(k, 1))
oracle.kv_release(pt, kv_len, nxt)
print("sanitized oracle run complete")
'''


def test_oracle_is_clean_under_asan_and_ubsan():
    try:
        asan = subprocess.check_output(["gcc", "-print-file-name=libasan.so"], text=True).strip()
    except Exception:
        pytest.skip("gcc not available")
    if not os.path.isabs(asan) or not os.path.exists(asan):
        pytest.skip("libasan not installed")
    env = dict(os.environ, FLEXSPEC_ORACLE_SANITIZE="1", LD_PRELOAD=asan, PYTHONPATH=ROOT,
               ASAN_OPTIONS="detect_leaks=0:halt_on_error=1:abort_on_error=0",
               UBSAN_OPTIONS="halt_on_error=1:print_stacktrace=1", OMP_NUM_THREADS="2")
    out = subprocess.run([sys.executable, "-c", DRIVER], env=env, cwd=ROOT, capture_output=True, text=True, timeout=600)
    text = out.stdout + out.stderr
    assert out.returncode == 0, text[-3000:]
    assert "sanitized oracle run complete" in out.stdout
    assert "AddressSanitizer" not in text and "runtime error" not in text, text[-3000:]
