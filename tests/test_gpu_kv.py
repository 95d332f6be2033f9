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


def test_kv_release_matches_oracle():
    """Pages past the rolled-back length go to the free list and leave the table: the same set per
    sequence, in the same order, as the oracle's (the order of the sequences in the list is free)."""
    import oracle
    from paper_2601_00644_b200 import binding as B
    rng = np.random.RandomState(77)
    batch, max_pages, num_pages = 37, 40, 2000
    prev = rng.randint(1, max_pages * 16 + 1, batch).astype(np.int32)
    nxt = np.array([rng.randint(1, p + 1) for p in prev], np.int32)
    nxt[3] = prev[3]                                       # nothing rejected
    ids = rng.permutation(num_pages).astype(np.int32)
    pt = np.full((batch, max_pages), -1, np.int32)
    c = 0
    for b in range(batch):
        n = -(-int(prev[b]) // 16)
        pt[b, :n] = ids[c:c + n]; c += n
    want_pt, want_free = oracle.kv_release(pt, prev, nxt)
    w = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    ver = B.Verifier(w, 1, 1, 64, max_batch=batch, k_max=1, max_kv_len=max_pages * 16)
    pt_d = torch.from_numpy(pt).cuda()
    free = torch.full((num_pages,), -7, dtype=torch.int32, device="cuda")
    count = torch.tensor([5], dtype=torch.int32, device="cuda")            # the list already holds five entries
    ver.kv_release(pt_d, num_pages, torch.from_numpy(prev).cuda(), torch.from_numpy(nxt).cuda(), free, count)
    torch.cuda.synchronize()
    assert ver.status()[0] == 0
    assert np.array_equal(pt_d.cpu().numpy(), want_pt)
    n_free = int(count.item()) - 5
    assert n_free == len(want_free)
    got = free.cpu().numpy()
    assert np.all(got[:5] == -7) and np.all(got[5 + n_free:] == -7)
    assert sorted(got[5:5 + n_free].tolist()) == sorted(want_free.tolist())
    # a sequence's pages are contiguous in the list and in ascending entry order
    pos = {int(p): i for i, p in enumerate(got[5:5 + n_free])}
    for b in range(batch):
        keep, had = -(-int(nxt[b]) // 16), -(-int(prev[b]) // 16)
        idx = [pos[int(p)] for p in pt[b, keep:had]]
        assert idx == list(range(idx[0], idx[0] + len(idx))) if idx else True
    # a list that is too short is reported, nothing is written past it
    pt_d = torch.from_numpy(pt).cuda()
    small = torch.full((3,), -7, dtype=torch.int32, device="cuda")
    count.zero_()
    ver.kv_release(pt_d, num_pages, torch.from_numpy(prev).cuda(), torch.from_numpy(nxt).cuda(), small, count)
    torch.cuda.synchronize()
    assert ver.status()[0] == B.ERR_INVALID_ARG
    ver.close()


def test_serving_loop_append_verify_rollback_release():
    """Three consecutive steps of one batch, as a serving loop would run them (Section IV-C and Algorithm 2):
    hand pages to the sequences that need them, append the window's K/V, verify, roll kv_len back,
    release the pages past it, draft again from the new length.  Every step's pool, attention output,
    decisions, lengths, page table and released pages are compared with the oracle run on the same state."""
    import tests.harness as H
    from paper_2601_00644_b200 import binding as B
    rng = np.random.RandomState(91)
    Hq, Hkv, Dh, V, batch, k_max = 8, 2, 64, 2048, 5, 4
    d = Hq * Dh
    max_pages = 12
    num_pages = batch * max_pages
    gen = torch.Generator(device="cuda").manual_seed(91)
    w = (torch.randn(V, d, generator=gen, device="cuda") * 0.05).to(torch.bfloat16)
    pool = torch.randn(num_pages, 2, Hkv, 16, Dh, generator=gen, device="cuda").to(torch.bfloat16)
    ver = B.Verifier(w, Hq, Hkv, Dh, max_batch=batch, k_max=k_max, max_kv_len=max_pages * 16, debug=True)
    pt_h = np.full((batch, max_pages), -1, np.int32)             # nobody owns a page yet
    free_h = rng.permutation(num_pages).astype(np.int32)         # the free list holds them all
    n_free = num_pages
    ctx = rng.randint(3, 60, batch).astype(np.int32)             # committed context per sequence
    seeds = torch.from_numpy(rng.randint(0, 2 ** 62, batch).astype(np.int64)).cuda()
    seeds_h = seeds.cpu().numpy().view(np.uint64)
    released_total = 0
    for step in range(3):
        k = rng.randint(0, k_max + 1, batch).astype(np.int32)
        kv_len = (ctx + k + 1).astype(np.int32)
        # the serving loop hands pages from the free list to the sequences whose window needs them
        for b in range(batch):
            for i in range(-(-int(kv_len[b]) // 16)):
                if pt_h[b, i] < 0:
                    n_free -= 1
                    pt_h[b, i] = free_h[n_free]
        pt = torch.from_numpy(pt_h).cuda()
        free = torch.from_numpy(free_h).cuda()
        free_n = torch.tensor([n_free], dtype=torch.int32, device="cuda")
        m, s = int(k.sum()) + batch, int(k.sum())
        hidden = torch.randn(m, d, generator=gen, device="cuda").to(torch.bfloat16)
        new_k = torch.randn(m, Hkv, Dh, generator=gen, device="cuda").to(torch.bfloat16)
        new_v = torch.randn(m, Hkv, Dh, generator=gen, device="cuda").to(torch.bfloat16)
        zd = torch.randn(max(s, 1), V, generator=gen, device="cuda")[:s] * 2
        toks = torch.from_numpy(rng.randint(0, V, s).astype(np.int32)).cuda()
        k_d, kv_d = torch.from_numpy(k).cuda(), torch.from_numpy(kv_len).cuda()
        pool_before = wl.bits_u16(pool)
        ver.kv_append(pool, pt, kv_d, torch.from_numpy(kv_len), new_k, new_v, k_d, torch.from_numpy(k))
        acc, nxt = ver.verify(pool, pt, kv_d, torch.from_numpy(kv_len), hidden, toks, zd, k_d, torch.from_numpy(k), seeds)
        kv_next = ver.kv_rollback(kv_d, k_d, acc)
        ver.kv_release(pt, num_pages, kv_d, kv_next, free, free_n)
        torch.cuda.synchronize()
        assert ver.status()[0] == 0
        # ---- the oracle on the same state
        want_pool = oracle.kv_append(pool_before, pt_h, kv_len, k, wl.bits_u16(new_k), wl.bits_u16(new_v), Hkv, Dh)
        assert np.array_equal(wl.bits_u16(pool), want_pool)
        ref = oracle.verify(oracle.SAMPLE, wl.bits_u16(hidden), want_pool, pt_h, kv_len, k, wl.bits_u16(w),
                            toks.cpu().numpy(), zd.cpu().numpy(), seeds_h, Hq, Hkv, Dh)
        dbg = ver.debug(m, s)
        err, ok = H.rel_close(dbg["attn_out"].float().cpu().numpy(), ref["attn_f64"])
        assert ok and err < H.REL_TOL
        iso = oracle.accept(oracle.SAMPLE, dbg["logits"].cpu().numpy().astype(np.float64), zd.cpu().numpy(), toks.cpu().numpy(),
                            k, seeds_h)
        acc_h, nxt_h = acc.cpu().numpy(), nxt.cpu().numpy()
        t0 = np.concatenate([[0], np.cumsum(k)])
        for b in range(batch):                                  # the oracle on the same logits: identical except at near-ties
            if acc_h[b] != iso["accepted_len"][b]:
                assert iso["acc_margin"][t0[b] + min(acc_h[b], iso["accepted_len"][b])] < H.TIE_TOL
            elif nxt_h[b] != iso["next_token"][b]:
                assert iso["cdf_margin"][b] < H.CDF_TIE_TOL
        kv_next_h = kv_next.cpu().numpy()
        assert np.array_equal(kv_next_h, oracle.kv_rollback(kv_len, k, acc_h))
        want_pt, want_freed = oracle.kv_release(pt_h, kv_len, kv_next_h)
        assert np.array_equal(pt.cpu().numpy(), want_pt)
        n_after = int(free_n.item())
        assert n_after - n_free == len(want_freed)
        assert sorted(free.cpu().numpy()[n_free:n_after].tolist()) == sorted(want_freed.tolist())
        released_total += len(want_freed)
        # the next step starts from the committed context + accepted drafts + the emitted token's position
        pt_h, free_h, n_free = want_pt, free.cpu().numpy(), n_after
        ctx = kv_next_h.astype(np.int32)
    # every page is either owned by exactly one sequence or on the free list
    owned = pt_h[pt_h >= 0]
    assert len(set(owned.tolist())) == len(owned)
    assert set(owned.tolist()).isdisjoint(set(free_h[:n_free].tolist())) and len(owned) + n_free == num_pages
    ver.close()
