"""GPU parity of the KV-session steps around verification (Section IV-C): append of the window's
K/V rows and the device-side rollback of kv_len, bit-exact against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_00644_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("kw", [
    dict(batch=1, n_q_heads=8, n_kv_heads=2, head_dim=64, k_min=4, k_max=4, ctx_min=128, ctx_max=128),
    dict(batch=7, n_q_heads=32, n_kv_heads=8, head_dim=128, k_min=0, k_max=12, ctx_min=0, ctx_max=900),
])
def test_kv_append_and_rollback_match_oracle(kw):
    from paper_2601_00644_b200 import binding as B
    shape = wl.VerifyShape(name="kv_case", index=300 + kw["batch"], vocab=256, sigma_min=0.5, sigma_max=0.5, **kw)
    inp = wl.make_inputs(shape, device="cuda", with_noise=False)
    k_host, kv_host = inp.draft_len.cpu(), inp.kv_len.cpu()
    ver = B.Verifier(inp.lm_head_w, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, max_batch=inp.batch,
                     k_max=max(int(k_host.max()), 1), max_kv_len=int(kv_host.max()))
    gen = torch.Generator(device="cuda").manual_seed(77)
    m = inp.m_rows
    new_k = torch.randn(m, shape.n_kv_heads, shape.head_dim, generator=gen, device="cuda").to(torch.bfloat16)
    new_v = torch.randn(m, shape.n_kv_heads, shape.head_dim, generator=gen, device="cuda").to(torch.bfloat16)
    pool = inp.kv_pages.clone()
    ver.kv_append(pool, inp.page_table, inp.kv_len, kv_host, new_k, new_v, inp.draft_len, k_host)
    torch.cuda.synchronize()
    assert ver.status()[0] == 0
    want = oracle.kv_append(wl.bits_u16(inp.kv_pages), inp.page_table.cpu().numpy(), kv_host.numpy(), k_host.numpy(),
                            wl.bits_u16(new_k), wl.bits_u16(new_v), shape.n_kv_heads, shape.head_dim)
    assert np.array_equal(wl.bits_u16(pool), want)                 # byte work: bit-exact
    # the appended rows are what attention reads
    out = ver.attention(pool, inp.page_table, inp.kv_len, kv_host, inp.hidden, inp.draft_len, k_host)
    a64, _ = oracle.attention(wl.bits_u16(inp.hidden), want, inp.page_table.cpu().numpy(), kv_host.numpy(), k_host.numpy(),
                              shape.n_q_heads, shape.n_kv_heads, shape.head_dim)
    got = out.float().cpu().numpy()
    assert np.abs(got - a64).max() <= 2e-2 * np.abs(a64).max()
    # rollback
    rng = np.random.RandomState(5)
    acc = np.array([rng.randint(0, kk + 1) for kk in k_host.numpy()], np.int32)
    nxt = ver.kv_rollback(inp.kv_len, inp.draft_len, torch.from_numpy(acc).cuda())
    assert np.array_equal(nxt.cpu().numpy(), oracle.kv_rollback(kv_host.numpy(), k_host.numpy(), acc))
    ver.close()
