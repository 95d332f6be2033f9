"""GPU parity of each stage in isolation, through the C ABI, against the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_00644_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _binding():
    from paper_2601_00644_b200 import binding
    return binding


def _rand_bf16(gen, shape, std):
    return (torch.randn(shape, generator=gen, device="cuda") * std).to(torch.bfloat16)


# ------------------------------------------------------------------ LM head

@pytest.mark.parametrize("m,d,v", [
    (5, 512, 4096),          # the tiny config's shape
    (1, 64, 128),            # smallest legal problem
    (96, 1024, 5000),        # ragged last vocabulary tile (5000 = 39*128 + 8)
    (100, 256, 777),         # vocab not a multiple of 4, rows not a multiple of 16
    (300, 512, 1300),        # two accumulator blocks (single TMEM buffer)
    (600, 256, 1000),        # two passes over W
    (40, 192, 20011),        # more tiles than SMs: full waves, then a wave of short tiles (re-tiled copy of W, both boxes)
    (530, 128, 19500),       # the same with two passes
])
def test_lm_head_matches_oracle(m, d, v):
    B = _binding()
    gen = torch.Generator(device="cuda").manual_seed(1000 + m)
    x = _rand_bf16(gen, (m, d), 1.0)
    w = _rand_bf16(gen, (v, d), 1.0)
    hd = 64
    ver = B.Verifier(w, d // hd, d // hd, hd, max_batch=max(m, 1), k_max=0, max_kv_len=16)
    logits = torch.full((m, v), float("nan"), device="cuda")
    ver.lm_head(x, logits)
    torch.cuda.synchronize()
    assert ver.status()[0] == 0
    ref = oracle.lm_head(wl.bits_u16(x), wl.bits_u16(w))
    got = logits.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    # fp32 accumulation of exact bf16 products: error ~ d * 2^-24 relative to sum |x||w|
    bound = d * 2.0 ** -23 * (np.abs(oracle.bf16_to_f64(wl.bits_u16(x))) @ np.abs(oracle.bf16_to_f64(wl.bits_u16(w))).T)
    assert np.all(np.abs(got - ref) <= bound + 1e-30)
    assert np.abs(got - ref).max() <= 2e-2 * np.abs(ref).max()
    # run-to-run determinism
    logits2 = torch.empty_like(logits)
    ver.lm_head(x, logits2)
    torch.cuda.synchronize()
    assert torch.equal(logits, logits2)
    ver.close()


# ------------------------------------------------------------------ attention

def _attn_parity(shape, tol=2e-2):
    import tests.harness as H
    case = H.Case(shape)
    ver = H.make_verifier(case)
    inp = case.inp
    out = ver.attention(inp.kv_pages, inp.page_table, inp.kv_len, inp.kv_len.cpu(), inp.hidden,
                        inp.draft_len, inp.draft_len.cpu())
    torch.cuda.synchronize()
    assert ver.status()[0] == 0
    s = shape
    a64, _ = oracle.attention(case.h_hidden, case.h_kv, case.h_pt, case.kv_len, case.k,
                              s.n_q_heads, s.n_kv_heads, s.head_dim)
    got = out.float().cpu().numpy()
    row_err, ok = H.rel_close(got, a64, tol)
    assert ok and row_err < tol, (row_err, ok)
    out2 = ver.attention(inp.kv_pages, inp.page_table, inp.kv_len, inp.kv_len.cpu(), inp.hidden,
                         inp.draft_len, inp.draft_len.cpu())
    torch.cuda.synchronize()
    assert torch.equal(out, out2)
    ver.close()
    return row_err


def _shape(name, idx, **kw):
    base = dict(batch=1, n_q_heads=8, n_kv_heads=2, head_dim=64, vocab=256, k_min=4, k_max=4,
                ctx_min=128, ctx_max=128, sigma_min=0.5, sigma_max=0.5)
    base.update(kw)
    return wl.VerifyShape(name=name, index=idx, **base)


@pytest.mark.parametrize("kw", [
    dict(),                                                              # tiny config: one split
    dict(input_std=1.0),                                                 # peaked scores
    dict(batch=5, k_min=0, k_max=12, ctx_min=1, ctx_max=700),            # ragged, several splits, k=0
    dict(batch=3, n_q_heads=32, n_kv_heads=8, head_dim=128, k_min=5, k_max=5, ctx_min=2048,
         ctx_max=2048, input_std=1.0),                                   # 8B heads
    dict(batch=2, n_q_heads=64, n_kv_heads=8, head_dim=128, k_min=8, k_max=8, ctx_min=1000,
         ctx_max=1300, input_std=1.0),                                   # 70B heads: 72 rows per kv head
    dict(batch=2, n_q_heads=32, n_kv_heads=8, head_dim=128, k_min=16, k_max=16, ctx_min=5000,
         ctx_max=6000, input_std=1.0),                                   # 68 rows, long context
    dict(batch=2, n_q_heads=16, n_kv_heads=1, head_dim=64, k_min=9, k_max=10, ctx_min=0,
         ctx_max=40, input_std=1.0),                                     # 176 rows per kv head: two row blocks
    dict(batch=4, n_q_heads=4, n_kv_heads=4, head_dim=128, k_min=1, k_max=3, ctx_min=0, ctx_max=3,
         input_std=1.0),                                                 # plain MHA, almost no context
])
def test_attention_matches_oracle(kw):
    _attn_parity(_shape("attn_case", 100 + len(kw), **kw))


# ------------------------------------------------------------------ decision stage

def _sample_case(seed, batch, vocab, k_lo, k_hi, mode, temperature, logit_std=3.0, holes=False, mask=False):
    rng = np.random.RandomState(seed)
    k = rng.randint(k_lo, k_hi + 1, batch).astype(np.int32)
    m, s = int(k.sum()) + batch, int(k.sum())
    zt = (rng.standard_normal((m, vocab)) * logit_std).astype(np.float32)
    zd = (rng.standard_normal((s, vocab)) * logit_std).astype(np.float32)
    # make the draft resemble the target so that acceptances and rejections both occur
    r0 = np.concatenate([[0], np.cumsum(k + 1)]); t0 = np.concatenate([[0], np.cumsum(k)])
    for b in range(batch):
        zd[t0[b]:t0[b + 1]] = zt[r0[b]:r0[b] + k[b]] + 0.7 * zd[t0[b]:t0[b + 1]] / logit_std
    if holes:
        zd[rng.rand(s, vocab) < 0.1] = -np.inf
        zt[rng.rand(m, vocab) < 0.05] = -np.inf
        zt[:, 0] = 1e4 * (rng.rand(m) < 0.1)                # a few rows with one huge logit
    q = torch.softmax(torch.from_numpy(zd).double() / max(temperature, 1e-3), -1).numpy() if s else np.zeros((0, vocab))
    toks = np.array([rng.choice(vocab, p=q[i] / q[i].sum()) for i in range(s)], np.int32)
    if mode == 1:      # greedy: make most drafts the arg-max so that prefixes get accepted
        am = np.concatenate([zt[r0[b]:r0[b] + k[b]].argmax(-1) for b in range(batch)]) if s else toks
        toks = np.where(rng.rand(s) < 0.7, am, toks).astype(np.int32)
    seeds = rng.randint(0, 2 ** 62, batch).astype(np.uint64)
    vmask = None
    if mask:
        vmask = rng.randint(0, 2 ** 32, (batch, (vocab + 31) // 32), dtype=np.uint64).astype(np.uint32)
        vmask[:, 0] |= 1
    return k, zt, zd, toks, seeds, vmask


@pytest.mark.parametrize("mode,temperature", [(0, 1.0), (0, 0.7), (1, 1.0), (0, 0.0)])
@pytest.mark.parametrize("vocab,batch,k_hi,holes,mask", [
    (4096, 3, 4, False, False),
    (777, 9, 7, True, False),            # vocab % 4 != 0, -inf entries, huge logits
    (20000, 16, 12, False, True),        # several chunks with a ragged last one, vocabulary mask
    (8192 * 2 + 1, 5, 33, False, False), # k > 32: two ballot rounds
])
def test_sample_stage_matches_oracle(mode, temperature, vocab, batch, k_hi, holes, mask):
    B = _binding()
    k, zt, zd, toks, seeds, vmask = _sample_case(vocab + batch, batch, vocab, 0, k_hi, mode, temperature,
                                                 holes=holes, mask=mask)
    greedy = (mode == 1 or temperature == 0.0)
    w = torch.zeros(vocab, 64, dtype=torch.bfloat16, device="cuda")
    ver = B.Verifier(w, 1, 1, 64, max_batch=batch, k_max=max(k_hi, 1), max_kv_len=64, mode=mode, debug=True)
    dev = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a)).to(dt).cuda()
    zt_d, zd_d = dev(zt, torch.float32), dev(zd, torch.float32)
    toks_d = dev(toks, torch.int32)
    k_d = dev(k, torch.int32)
    seeds_d = dev(seeds.view(np.int64), torch.int64)
    vm_d = None if vmask is None else dev(vmask.view(np.int32), torch.int32)
    outs = []
    for _ in range(2):                   # twice: the self-resetting tickets must be reusable
        acc, nxt = ver.sample(zt_d, toks_d, zd_d, k_d, k_d.cpu(), seeds_d, temperature=temperature, vocab_mask=vm_d)
        torch.cuda.synchronize()
        assert ver.status()[0] == 0
        outs.append((acc.cpu().numpy(), nxt.cpu().numpy()))
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])
    acc, nxt = outs[0]
    ref = oracle.accept(1 if greedy else 0, zt.astype(np.float64), zd, toks, k, seeds,
                        temperature if not greedy else 1.0, vmask)
    t0 = np.concatenate([[0], np.cumsum(k)])
    n_ties = 0
    for b in range(batch):
        if acc[b] != ref["accepted_len"][b]:
            assert not greedy
            j = min(acc[b], ref["accepted_len"][b])
            assert ref["acc_margin"][t0[b] + j] < 1e-5
            n_ties += 1
            continue
        if nxt[b] != ref["next_token"][b]:
            assert not greedy and ref["cdf_margin"][b] < 1e-6, (b, nxt[b], ref["next_token"][b], ref["cdf_margin"][b])
    assert n_ties <= 1
    if not greedy and k.sum() > 0:
        dbg = ver.debug(int(k.sum()) + batch, int(k.sum()))
        assert np.abs(dbg["p_tok"].cpu().numpy() - ref["p_tok"]).max() < 1e-5
        assert np.abs(dbg["q_tok"].cpu().numpy() - ref["q_tok"]).max() < 1e-5
        assert np.array_equal(dbg["u"].cpu().numpy().astype(np.float64), ref["u"])
    ver.close()


def test_sample_invariants_on_gpu():
    """p == q accepts every draft; a draft outside the target's support is rejected at 0."""
    B = _binding()
    vocab, batch, kk = 5000, 6, 5
    rng = np.random.RandomState(5)
    k = np.full(batch, kk, np.int32)
    zt = (rng.standard_normal((batch * (kk + 1), vocab)) * 2).astype(np.float32)
    zd = zt.reshape(batch, kk + 1, vocab)[:, :kk].reshape(-1, vocab).copy()
    toks = rng.randint(0, vocab, batch * kk).astype(np.int32)
    seeds = rng.randint(0, 2 ** 62, batch).astype(np.int64)
    w = torch.zeros(vocab, 64, dtype=torch.bfloat16, device="cuda")
    ver = B.Verifier(w, 1, 1, 64, max_batch=batch, k_max=kk, max_kv_len=64)
    t = lambda a, dt: torch.from_numpy(a).to(dt).cuda()
    acc, nxt = ver.sample(t(zt, torch.float32), t(toks, torch.int32), t(zd, torch.float32), t(k, torch.int32),
                          torch.from_numpy(k), t(seeds, torch.int64), temperature=0.7)
    assert np.all(acc.cpu().numpy() == kk)
    # disjoint support through the vocabulary mask: drafts live on masked tokens only
    toks2 = (rng.randint(0, vocab // 2, batch * kk) * 2 + 1).astype(np.int32)          # odd ids
    words = (vocab + 31) // 32
    mask = np.full((batch, words), 0x55555555, np.uint32)                               # even ids allowed
    acc, nxt = ver.sample(t(zt, torch.float32), t(toks2, torch.int32), t(zd, torch.float32), t(k, torch.int32),
                          torch.from_numpy(k), t(seeds, torch.int64), temperature=0.7,
                          vocab_mask=t(mask.view(np.int32), torch.int32))
    assert np.all(acc.cpu().numpy() == 0)
    assert np.all(nxt.cpu().numpy() % 2 == 0)
    ver.close()


# ------------------------------------------------------------------ nucleus (top-p) sampling

@pytest.mark.parametrize("top_p,temperature", [(0.9, 1.0), (0.5, 0.7), (0.999, 1.0)])
@pytest.mark.parametrize("vocab,batch,k_hi,holes,mask", [
    (4096, 3, 4, False, False),
    (777, 9, 7, True, False),
    (20000, 16, 12, False, True),
])
def test_sample_stage_with_top_p_matches_oracle(top_p, temperature, vocab, batch, k_hi, holes, mask):
    B = _binding()
    k, zt, zd, toks, seeds, vmask = _sample_case(7 * vocab + batch, batch, vocab, 0, k_hi, 0, temperature,
                                                 holes=holes, mask=mask)
    w = torch.zeros(vocab, 64, dtype=torch.bfloat16, device="cuda")
    ver = B.Verifier(w, 1, 1, 64, max_batch=batch, k_max=max(k_hi, 1), max_kv_len=64, mode=0, debug=True)
    ver.set_top_p(top_p)
    dev = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a)).to(dt).cuda()
    vm_d = None if vmask is None else dev(vmask.view(np.int32), torch.int32)
    acc, nxt = ver.sample(dev(zt, torch.float32), dev(toks, torch.int32), dev(zd, torch.float32), dev(k, torch.int32),
                          torch.from_numpy(k), dev(seeds.view(np.int64), torch.int64), temperature=temperature, vocab_mask=vm_d)
    torch.cuda.synchronize()
    assert ver.status()[0] == 0
    acc, nxt = acc.cpu().numpy(), nxt.cpu().numpy()
    ref = oracle.accept(0, zt.astype(np.float64), zd, toks, k, seeds, temperature, vmask, top_p=top_p)
    r0 = np.concatenate([[0], np.cumsum(k + 1)]); t0 = np.concatenate([[0], np.cumsum(k)])
    dbg = ver.debug(int(k.sum()) + batch, int(k.sum()))
    p_g = dbg["p_tok"].cpu().numpy()
    excused = 0
    for b in range(batch):
        kb = int(k[b])
        # a nucleus cut that falls within 1e-6 of top_p may legitimately land one token earlier / later:
        # only then may an outcome differ beyond the usual near-tie clauses
        cut_tie = ref["topp_margin"][r0[b]:r0[b + 1]].min() < 1e-6
        bad = False
        if kb and np.abs(p_g[t0[b]:t0[b] + kb] - ref["p_tok"][t0[b]:t0[b] + kb]).max() >= 1e-5:
            bad = True
        elif acc[b] != ref["accepted_len"][b]:
            j = min(acc[b], ref["accepted_len"][b])
            if ref["acc_margin"][t0[b] + j] < 1e-5:
                excused += 1
                continue
            bad = True
        elif nxt[b] != ref["next_token"][b] and not ref["cdf_margin"][b] < 1e-6:
            bad = True
        if bad:
            assert cut_tie, (b, acc[b], ref["accepted_len"][b], nxt[b], ref["next_token"][b])
            excused += 1
    assert excused <= 1
    # the filter is really on: with top_p = 0.5 some draft token fell outside its row's nucleus
    if top_p == 0.5 and k.sum() > 0:
        assert (ref["p_tok"] == 0).any() and (p_g[ref["p_tok"] == 0] == 0).all()
    ver.set_top_p(1.0)
    acc1, nxt1 = ver.sample(dev(zt, torch.float32), dev(toks, torch.int32), dev(zd, torch.float32), dev(k, torch.int32),
                            torch.from_numpy(k), dev(seeds.view(np.int64), torch.int64), temperature=temperature, vocab_mask=vm_d)
    ref1 = oracle.accept(0, zt.astype(np.float64), zd, toks, k, seeds, temperature, vmask)
    assert (acc1.cpu().numpy() != ref1["accepted_len"]).sum() <= 1           # switched off again
    ver.close()


def test_device_lengths_that_disagree_with_the_host_copy_are_reported():
    """The launches are sized from draft_len_host; the kernels index with the device copy.  A device
    copy that disagrees must not send any index outside its array: the row-offset kernel reports
    INVALID_ARG through the status word and the stage runs with every k_b = 0."""
    from paper_2601_00644_b200 import binding as B
    rng = np.random.RandomState(3)
    batch, vocab = 5, 4096
    k = np.array([2, 0, 3, 1, 2], np.int32)
    m, s = int(k.sum()) + batch, int(k.sum())
    zt = torch.from_numpy(rng.standard_normal((m, vocab)).astype(np.float32)).cuda()
    zd = torch.from_numpy(rng.standard_normal((s, vocab)).astype(np.float32)).cuda()
    toks = torch.from_numpy(rng.randint(0, vocab, s).astype(np.int32)).cuda()
    seeds = torch.from_numpy(rng.randint(0, 2 ** 62, batch).astype(np.int64)).cuda()
    w = torch.zeros(vocab, 64, dtype=torch.bfloat16, device="cuda")
    ver = B.Verifier(w, 1, 1, 64, max_batch=batch, k_max=8, max_kv_len=64)
    for bad in ([2, 0, 4, 1, 2], [2, 0, 3, 1, 1], [2, -1, 3, 1, 2], [2, 0, 7, 0, 0]):
        k_dev = torch.tensor(bad, dtype=torch.int32, device="cuda")
        acc, nxt = ver.sample(zt, toks, zd, k_dev, torch.from_numpy(k), seeds)
        torch.cuda.synchronize()
        code, st = ver.status()
        assert code == B.ERR_INVALID_ARG, (bad, code, st)
        assert torch.all(acc == 0) and torch.all((nxt >= 0) & (nxt < vocab))
    # and the handle is fine afterwards
    acc, nxt = ver.sample(zt, toks, zd, torch.from_numpy(k).cuda(), torch.from_numpy(k), seeds)
    torch.cuda.synchronize()
    assert ver.status()[0] == 0 and torch.all((acc >= 0) & (acc <= torch.from_numpy(k).cuda()))
    ver.close()


def test_a_bounded_wait_runs_out_and_is_reported():
    """The wait routine of every pipeline, on a barrier nobody signals, with a limit of two
    milliseconds: the kernel returns by itself, the status word holds the timeout, and the handle
    goes on working."""
    import time
    from paper_2601_00644_b200 import binding as B
    w = torch.zeros(256, 64, dtype=torch.bfloat16, device="cuda")
    ver = B.Verifier(w, 1, 1, 64, max_batch=1, k_max=1, max_kv_len=64)
    t0 = time.perf_counter()
    ver.selftest_wait_timeout(2_000_000)
    torch.cuda.synchronize()
    waited = time.perf_counter() - t0
    code, st = ver.status()
    assert code == B.ERR_TIMEOUT and st[2] == 99
    assert 0.0015 < waited < 1.0
    assert ver.status()[0] == 0                    # cleared by the read
    with pytest.raises(B.FlexSpecError):
        ver.selftest_wait_timeout(10 ** 9)         # limits beyond 50 ms are refused on the host
    ver.close()


# ------------------------------------------------------------------ top-k and per-sequence temperatures

def _decisions_match(k, acc, nxt, ref, p_g=None, skip=()):
    """Identical decisions except at near-ties (1e-5 acceptance, 1e-6 inverse CDF); returns #excused."""
    t0 = np.concatenate([[0], np.cumsum(k)])
    excused = 0
    for b in range(len(k)):
        if b in skip:
            continue
        kb = int(k[b])
        if p_g is not None and kb:
            assert np.abs(p_g[t0[b]:t0[b] + kb] - ref["p_tok"][t0[b]:t0[b] + kb]).max() < 1e-5, b
        if acc[b] != ref["accepted_len"][b]:
            assert ref["acc_margin"][t0[b] + min(acc[b], ref["accepted_len"][b])] < 1e-5, b
            excused += 1
        elif nxt[b] != ref["next_token"][b]:
            assert ref["cdf_margin"][b] < 1e-6, (b, nxt[b], ref["next_token"][b])
            excused += 1
    return excused


@pytest.mark.parametrize("top_k,top_p", [(1, 1.0), (5, 1.0), (50, 1.0), (40, 0.9), (3, 0.5)])
@pytest.mark.parametrize("vocab,batch,k_hi,holes,mask", [
    (4096, 3, 4, False, False),
    (777, 9, 7, True, False),
    (20000, 12, 12, False, True),
])
def test_sample_stage_with_top_k_matches_oracle(top_k, top_p, vocab, batch, k_hi, holes, mask):
    B = _binding()
    temperature = 0.8
    k, zt, zd, toks, seeds, vmask = _sample_case(11 * vocab + batch + top_k, batch, vocab, 0, k_hi, 0, temperature,
                                                 holes=holes, mask=mask)
    w = torch.zeros(vocab, 64, dtype=torch.bfloat16, device="cuda")
    ver = B.Verifier(w, 1, 1, 64, max_batch=batch, k_max=max(k_hi, 1), max_kv_len=64, mode=0, debug=True)
    ver.set_sampling(top_p=top_p, top_k=top_k)
    dev = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a)).to(dt).cuda()
    vm_d = None if vmask is None else dev(vmask.view(np.int32), torch.int32)
    acc, nxt = ver.sample(dev(zt, torch.float32), dev(toks, torch.int32), dev(zd, torch.float32), dev(k, torch.int32),
                          torch.from_numpy(k), dev(seeds.view(np.int64), torch.int64), temperature=temperature, vocab_mask=vm_d)
    torch.cuda.synchronize()
    assert ver.status()[0] == 0
    ref = oracle.accept(0, zt.astype(np.float64), zd, toks, k, seeds, temperature, vmask, top_p=top_p, top_k=top_k)
    r0 = np.concatenate([[0], np.cumsum(k + 1)])
    dbg = ver.debug(int(k.sum()) + batch, int(k.sum()))
    # a nucleus cut within 1e-6 of top_p may land one token earlier / later: such sequences are left out
    skip = [b for b in range(batch) if ref["topp_margin"][r0[b]:r0[b + 1]].min() < 1e-6]
    assert len(skip) <= 1
    assert _decisions_match(k, acc.cpu().numpy(), nxt.cpu().numpy(), ref, dbg["p_tok"].cpu().numpy(), skip) <= 1
    if top_k <= 5 and k.sum() > 0:                    # the filter is really on
        assert (ref["p_tok"] == 0).any()
    ver.close()


def test_sample_stage_with_per_sequence_temperatures_matches_oracle():
    B = _binding()
    batch, vocab, k_hi = 10, 6000, 6
    k, zt, zd, toks, seeds, _ = _sample_case(4242, batch, vocab, 0, k_hi, 0, 1.0)
    temps = np.array([0.5, 1.0, 0.7, 1.3, 2.0, 0.9, 1.0, 0.6, 1.7, 0.8], np.float32)
    w = torch.zeros(vocab, 64, dtype=torch.bfloat16, device="cuda")
    ver = B.Verifier(w, 1, 1, 64, max_batch=batch, k_max=k_hi, max_kv_len=64, mode=0, debug=True)
    dev = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a)).to(dt).cuda()
    args = (dev(zt, torch.float32), dev(toks, torch.int32), dev(zd, torch.float32), dev(k, torch.int32),
            torch.from_numpy(k), dev(seeds.view(np.int64), torch.int64))
    for top_p, top_k in [(1.0, 0), (0.9, 30)]:
        ver.set_sampling(top_p=top_p, top_k=top_k, temperatures=dev(temps, torch.float32))
        acc, nxt = ver.sample(*args, temperature=1.0)          # the scalar is overridden per sequence
        torch.cuda.synchronize()
        assert ver.status()[0] == 0
        ref = oracle.accept(0, zt.astype(np.float64), zd, toks, k, seeds, 1.0, None, top_p=top_p, top_k=top_k,
                            temperatures=temps.astype(np.float64))
        r0 = np.concatenate([[0], np.cumsum(k + 1)])
        skip = [b for b in range(batch) if ref["topp_margin"][r0[b]:r0[b + 1]].min() < 1e-6]
        dbg = ver.debug(int(k.sum()) + batch, int(k.sum()))
        assert _decisions_match(k, acc.cpu().numpy(), nxt.cpu().numpy(), ref, dbg["p_tok"].cpu().numpy(), skip) <= 1
    # a temperature that is not a positive finite number is reported, and the scalar is used for that sequence
    bad = temps.copy(); bad[3] = 0.0
    ver.set_sampling(temperatures=dev(bad, torch.float32))
    ver.sample(*args, temperature=1.0)
    torch.cuda.synchronize()
    assert ver.status()[0] == B.ERR_INVALID_ARG
    # switched off again: the scalar applies to every sequence
    ver.set_sampling()
    acc, nxt = ver.sample(*args, temperature=0.9)
    ref = oracle.accept(0, zt.astype(np.float64), zd, toks, k, seeds, 0.9)
    assert _decisions_match(k, acc.cpu().numpy(), nxt.cpu().numpy(), ref) <= 1
    ver.close()


def test_stage_outputs_stay_inside_their_buffers():
    """Attention output and logits written into caller buffers that sit between canary guard bands
    (ragged batch: the last query row and the last vocabulary tile are partial): the bands survive."""
    import tests.harness as H
    B = _binding()
    shape = _shape("guard", 31, batch=3, n_q_heads=8, n_kv_heads=2, head_dim=128, vocab=1000 + 37, k_min=0, k_max=6,
                   ctx_min=5, ctx_max=300)
    inp = wl.make_inputs(shape, device="cuda")
    kh, kvh = inp.draft_len.cpu(), inp.kv_len.cpu()
    ver = B.Verifier(inp.lm_head_w, 8, 2, 128, max_batch=3, k_max=6, max_kv_len=int(kvh.max()))
    m, d, v = inp.m_rows, shape.d_model, shape.vocab
    a_w, a = H.guarded(m * d, torch.bfloat16)
    ver.attention(inp.kv_pages, inp.page_table, inp.kv_len, kvh, inp.hidden, inp.draft_len, kh, attn_out=a.view(m, d))
    l_w, l = H.guarded(m * v, torch.float32)
    ver.lm_head(a.view(m, d), logits=l.view(m, v))
    torch.cuda.synchronize()
    assert ver.status()[0] == 0
    assert H.guards_intact(a_w, m * d) and H.guards_intact(l_w, m * v)
    assert int((l.view(torch.int32) == H.CANARY).sum()) == 0                # and everything inside was written
    ver.close()


# ------------------------------------------------------------------ attention over a sweep of seeded shapes

def _random_attention_shapes():
    """Seeded shapes that walk through every kernel instance and both cuts of the work list: head dims 64 / 128,
    group sizes 1..16, tiles of 1..128 query rows (one, two or three threads per token, single P^T buffer),
    contexts from empty to several blocks per CTA, batches from one sequence to more pairs than SMs."""
    rng = np.random.RandomState(20260106)
    shapes = []
    for i in range(14):
        head_dim = int(rng.choice([64, 128]))
        n_kv = int(rng.choice([1, 2, 4, 8]))
        group = int(rng.choice([1, 2, 4, 8, 16]))
        k_hi = int(rng.choice([0, 1, 3, 7, 12, 20]))
        k_hi = min(k_hi, 128 // group * 2)                 # up to two row blocks per kv head
        ctx_hi = int(rng.choice([0, 50, 400, 1500, 4000]))
        batch = int(rng.choice([1, 2, 5, 24]))
        if batch * ctx_hi * n_kv * head_dim > 24 * 1500 * 8 * 64:   # keep the oracle within a second or two
            ctx_hi = 400
        shapes.append(dict(batch=batch, n_q_heads=n_kv * group, n_kv_heads=n_kv, head_dim=head_dim, k_min=0, k_max=k_hi,
                           ctx_min=0, ctx_max=ctx_hi, input_std=float(rng.choice([0.02, 1.0])), idx=400 + i))
    return shapes


@pytest.mark.parametrize("kw", _random_attention_shapes(), ids=lambda kw: "b%dh%dx%dd%dk%dc%d" % (
    kw["batch"], kw["n_kv_heads"], kw["n_q_heads"] // kw["n_kv_heads"], kw["head_dim"], kw["k_max"], kw["ctx_max"]))
def test_attention_sweep_matches_oracle(kw):
    kw = dict(kw)
    idx = kw.pop("idx")
    _attn_parity(_shape("att_sweep", idx, **kw))


# ------------------------------------------------------------------ the filter's thresholds themselves

def _filter_rows(vocab, seed):
    """Rows that stress every path of the selection: ties by the thousand, one dominant token, duplicates
    around the cut, a spread of 1e-4, -inf entries, a heavy tail, plain normal rows."""
    rng = np.random.RandomState(seed)
    rows = [
        np.zeros(vocab),                                                     # all equal: one code, one logit value
        (rng.rand(vocab) < 0.5).astype(np.float64),                          # two values
        np.where(np.arange(vocab) == vocab // 3, 30.0, rng.standard_normal(vocab)),   # one dominant token
        np.round(rng.standard_normal(vocab) * 2.0 * 4.0) / 4.0,              # multiples of 0.25: many exact duplicates
        rng.standard_normal(vocab),
        rng.standard_normal(vocab) * 1e-4,                                   # flatter than any window guess
        np.where(rng.rand(vocab) < 0.2, -np.inf, rng.standard_normal(vocab)),
        rng.exponential(5.0, vocab),                                         # heavy upper tail
        rng.standard_normal(vocab) * 3.0 + 100.0,                            # large offset: coarse float grid
        -rng.exponential(0.01, vocab),                                       # most entries a hair below the maximum
    ]
    return np.stack(rows).astype(np.float32)


@pytest.mark.parametrize("top_p,top_k,temperature", [(0.9, 0, 1.0), (0.5, 0, 0.7), (0.999, 0, 1.0), (1.0, 1, 1.0),
                                                      (1.0, 7, 1.0), (0.9, 50, 1.3), (1.0, 900, 1.0), (0.3, 3, 1.0)])
@pytest.mark.parametrize("vocab", [1000, 1003, 32000, 140003])
def test_filter_thresholds_match_their_definition(top_p, top_k, temperature, vocab):
    """The lowest kept logit and the kept mass that the filter kernel leaves per row, against the definition
    (sorted prefix in fp64 through the oracle's top-k / nucleus routines) on the same fp32 logits."""
    B = _binding()
    zt = _filter_rows(vocab, 13 * vocab + top_k)
    rows = zt.shape[0]
    k = np.zeros(rows, np.int32)
    w = torch.zeros(vocab, 64, dtype=torch.bfloat16, device="cuda")
    ver = B.Verifier(w, 1, 1, 64, max_batch=rows, k_max=1, max_kv_len=64, mode=0, debug=True)
    ver.set_sampling(top_p=top_p, top_k=top_k)
    dev = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a)).to(dt).cuda()
    seeds = np.arange(1, rows + 1, dtype=np.int64)
    acc, nxt = ver.sample(dev(zt, torch.float32), dev(np.zeros(0, np.int32), torch.int32),
                          dev(np.zeros((0, vocab), np.float32), torch.float32), dev(k, torch.int32),
                          torch.from_numpy(k), dev(seeds, torch.int64), temperature=temperature)
    torch.cuda.synchronize()
    assert ver.status()[0] == 0
    got = ver.debug(rows, 0)["topp"].cpu().numpy()
    nxt = nxt.cpu().numpy()
    checked = 0
    for r in range(rows):
        z = zt[r].astype(np.float64)
        e = np.exp((z - z.max()) / temperature)
        p = e / e.sum()
        if 0 < top_k < vocab:
            p = oracle.topk(p, top_k)
        pk = p.copy()                                                        # the distribution the nucleus is cut from
        margin = np.inf
        if top_p < 1.0:
            p, margin = oracle.nucleus(p, top_p)
        kept = p > 0
        assert kept[nxt[r]], (r, "emitted token outside the kept set")
        kept_g = (z >= got[r, 0]) & np.isfinite(z)
        if margin < 1e-6:
            # the cut itself is a near-tie: the kernel's set must still be a minimal prefix within that slack
            assert kept_g[pk > 0].any() and not kept_g[pk == 0].any(), r
            assert pk[kept_g].sum() >= top_p - 2e-6 and pk[z > got[r, 0]].sum() < top_p + 2e-6, (r, pk[kept_g].sum())
            continue
        # the threshold is unique up to the gap below the lowest kept logit: compare the sets it defines
        assert np.array_equal(kept_g, kept), (r, got[r, 0], z[kept].min(), int(kept.sum()), int(kept_g.sum()))
        if kept.sum() < np.isfinite(z).sum():
            assert got[r, 0] == z[kept].min(), (r, got[r, 0], z[kept].min())  # and it is the lowest kept logit itself
        assert abs(got[r, 1] - e[kept].sum()) <= 2e-6 * e[kept].sum(), (r, got[r, 1], e[kept].sum())
        checked += 1
    assert checked >= 2
    ver.close()
