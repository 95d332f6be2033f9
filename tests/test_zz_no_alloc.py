"""flexspec_sample_static -- the entry point for hosts that cannot allocate device memory when
they call the library (their memory pool owns the device, or their step loop must not hit the
synchronisation an allocation implies).  It must give exactly what flexspec_sample gives; its
scratch is one array shared by all calls, so it is called twice in a row here, with inputs of
different sizes, to show that nothing left over from one call disturbs the next.

This file sorts last on purpose: a run that stops at the first failure has then already run
every other test."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _case(seed, batch, vocab, k_hi, temperature):
    rng = np.random.RandomState(seed)
    k = rng.randint(0, k_hi + 1, batch).astype(np.int32)
    m, s = int(k.sum()) + batch, int(k.sum())
    zt = (rng.standard_normal((m, vocab)) * 3).astype(np.float32)
    zd = (rng.standard_normal((s, vocab)) * 0.7).astype(np.float32)
    r0 = np.concatenate([[0], np.cumsum(k + 1)])
    t0 = np.concatenate([[0], np.cumsum(k)])
    for b in range(batch):                       # draft = target + noise: accepts and rejects both occur
        zd[t0[b]:t0[b + 1]] += zt[r0[b]:r0[b] + k[b]]
    q = torch.softmax(torch.from_numpy(zd).double() / temperature, -1).numpy() if s else np.zeros((0, vocab))
    toks = np.array([rng.choice(vocab, p=q[i] / q[i].sum()) for i in range(s)], np.int32)
    seeds = rng.randint(0, 2 ** 62, batch).astype(np.int64)
    dev = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a)).to(dt).cuda()
    return dict(k=k, zt=dev(zt, torch.float32), zd=dev(zd, torch.float32), toks=dev(toks, torch.int32),
                k_d=dev(k, torch.int32), k_h=torch.from_numpy(k), seeds=dev(seeds, torch.int64))


@pytest.mark.parametrize("mode,temperature", [(0, 1.0), (0, 0.7), (1, 1.0)])
def test_static_entry_matches_handle_entry_on_two_calls_in_a_row(mode, temperature):
    from paper_2601_00644_b200 import binding as B
    cases = [_case(71, 9, 20000, 7, temperature), _case(72, 4, 5001, 12, temperature)]
    for c in cases:                               # two calls in a row through the static entry point
        w = torch.zeros(c["zt"].shape[1], 64, dtype=torch.bfloat16, device="cuda")
        ver = B.Verifier(w, 1, 1, 64, max_batch=len(c["k"]), k_max=max(int(c["k"].max()), 1), max_kv_len=64, mode=mode)
        want_acc, want_nxt = ver.sample(c["zt"], c["toks"], c["zd"], c["k_d"], c["k_h"], c["seeds"],
                                        temperature=temperature)
        torch.cuda.synchronize()
        got_acc = torch.full_like(want_acc, -7)
        got_nxt = torch.full_like(want_nxt, -7)
        B.sample_static(c["zt"], c["toks"], c["zd"], c["k_d"], c["k_h"], c["seeds"], mode=mode,
                        temperature=temperature, accepted_len=got_acc, next_token=got_nxt)
        torch.cuda.synchronize()
        # integer outputs of the same arithmetic: the tolerance of the other decision tests is "identical"
        assert torch.equal(got_acc, want_acc)
        assert torch.equal(got_nxt, want_nxt)
        ver.close()
        # ... and against the fp64 oracle on the same logits: identical except at near-ties
        # (|u - min(1, p/q)| < 1e-5 for an acceptance test, 1e-6 for the inverse-CDF boundary)
        import oracle
        ref = oracle.accept(mode, c["zt"].cpu().numpy().astype(np.float64), c["zd"].cpu().numpy(),
                            c["toks"].cpu().numpy(), c["k"], c["seeds"].cpu().numpy().view(np.uint64), temperature)
        t0 = np.concatenate([[0], np.cumsum(c["k"])])
        acc, nxt = got_acc.cpu().numpy(), got_nxt.cpu().numpy()
        ties = 0
        for b in range(len(c["k"])):
            if acc[b] != ref["accepted_len"][b]:
                assert ref["acc_margin"][t0[b] + min(acc[b], ref["accepted_len"][b])] < 1e-5
                ties += 1
            elif nxt[b] != ref["next_token"][b]:
                assert ref["cdf_margin"][b] < 1e-6
                ties += 1
        assert ties <= 1


def test_static_entry_rejects_sizes_beyond_its_array():
    from paper_2601_00644_b200 import binding as B
    z = torch.zeros(1, 8, device="cuda")
    k_h = torch.zeros(65, dtype=torch.int32)      # batch 65 > 64
    with pytest.raises(B.FlexSpecError) as e:
        B.sample_static(z, None, None, k_h.cuda(), k_h, torch.zeros(65, dtype=torch.int64, device="cuda"))
    assert e.value.code == B.ERR_UNSUPPORTED
    k_h = torch.full((20,), 63, dtype=torch.int32)  # 20 * 64 rows > 1024
    with pytest.raises(B.FlexSpecError) as e:
        B.sample_static(z, torch.zeros(1260, dtype=torch.int32, device="cuda"), torch.zeros(1, 8, device="cuda"),
                        k_h.cuda(), k_h, torch.zeros(20, dtype=torch.int64, device="cuda"))
    assert e.value.code == B.ERR_UNSUPPORTED
