"""CPU pins for the fp64 oracle: every stage is checked against something other
than the oracle itself -- published known-answer vectors, dense brute force,
library fp64 routines, closed forms and the lossless property of the
speculative-sampling rule (Section II-A: outputs distributed exactly as the
target model's)."""
import math
import os

import numpy as np
import pytest
import scipy.special
import scipy.stats
import torch

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ bf16

def test_bf16_decode_encode_roundtrip_all_patterns():
    bits = np.arange(65536, dtype=np.uint16)
    with np.errstate(invalid="ignore"):
        vals = oracle.bf16_to_f64(bits)
    finite = np.isfinite(vals)
    back = oracle.f64_to_bf16(vals[finite])
    assert np.array_equal(back, bits[finite])


def test_bf16_encode_matches_fp32_rne_and_avoids_double_rounding():
    rng = np.random.RandomState(1)
    x32 = (rng.standard_normal(20000) * np.exp(rng.uniform(-20, 20, 20000))).astype(np.float32)
    want = torch.from_numpy(x32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = oracle.f64_to_bf16(x32.astype(np.float64))
    assert np.array_equal(got, want)
    # ties go to even
    assert oracle.f64_to_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 0x3F80          # -> 1.0
    assert oracle.f64_to_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 0x3F82      # -> 1 + 2^-6
    # just above a tie must round up although fp32 would first drop the excess
    assert oracle.f64_to_bf16(np.array([1.0 + 2.0 ** -8 + 2.0 ** -40]))[0] == 0x3F81
    assert oracle.f64_to_bf16(np.array([-(1.0 + 2.0 ** -8 + 2.0 ** -40)]))[0] == 0xBF81


# ---------------------------------------------------------------- Philox

def _kat():
    rows = []
    with open(os.path.join(GOLD, "philox4x32_10_kat.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            w = [int(t, 16) for t in line.split()]
            rows.append((w[0:4], w[4:6], w[6:10]))
    return rows


def test_philox_known_answers():
    rows = _kat()
    assert len(rows) == 3
    for ctr, key, out in rows:
        assert [int(v) for v in oracle.philox4x32_10(ctr, key)] == out


def test_uniform_convention_and_moments():
    seed = 0x0123456789ABCDEF
    for j, s in [(0, 0), (3, 1), (11, 0)]:
        w = oracle.philox4x32_10([j, s, 0, 0], [seed & 0xFFFFFFFF, seed >> 32])
        assert oracle.uniform(seed, j, s) == (int(w[0]) >> 8) / 2.0 ** 24
    u = np.array([oracle.uniform(77, j, 0) for j in range(100000)])
    assert u.min() >= 0.0 and u.max() < 1.0
    assert np.all(u * 2 ** 24 == np.round(u * 2 ** 24))
    assert abs(u.mean() - 0.5) < 4 * math.sqrt(1 / 12 / u.size)
    assert abs(u.var() - 1 / 12) < 2e-3
    # streams and seeds decorrelate
    v = np.array([oracle.uniform(77, j, 1) for j in range(100000)])
    assert abs(np.corrcoef(u, v)[0, 1]) < 0.02


# ------------------------------------------------------------- attention

def _rand_bf16(rng, shape, std=1.0):
    x = torch.from_numpy((rng.standard_normal(shape) * std).astype(np.float32)).to(torch.bfloat16)
    return x.view(torch.int16).numpy().view(np.uint16)


def _attn_case(rng, batch, hq, hkv, dh, k_list, ctx_list, page=16, std=1.0):
    k = np.array(k_list, np.int32)
    ctx = np.array(ctx_list, np.int32)
    kv_len = ctx + k + 1
    npages = (kv_len + page - 1) // page
    total = int(npages.sum()) + 2
    perm = rng.permutation(total).astype(np.int32)
    pt = np.full((batch, int(npages.max())), -1, np.int32)
    c = 0
    for b in range(batch):
        pt[b, :npages[b]] = perm[c:c + npages[b]]
        c += npages[b]
    m = int(k.sum()) + batch
    hidden = _rand_bf16(rng, (m, hq * dh), std)
    kv = _rand_bf16(rng, (total, 2, hkv, page, dh), std)
    return hidden, kv, pt, kv_len.astype(np.int32), k


def _dense_attention(hidden, kv, pt, kv_len, k, hq, hkv, dh, page=16):
    """Brute force: gather each sequence's K/V densely, full score matrix, explicit mask."""
    hid = oracle.bf16_to_f64(hidden)
    kvf = oracle.bf16_to_f64(kv)
    out = np.zeros_like(hid)
    g = hq // hkv
    r0 = 0
    for b in range(len(k)):
        L = int(kv_len[b])
        pages = pt[b, :(L + page - 1) // page]
        K = kvf[pages, 0].transpose(1, 0, 2, 3).reshape(hkv, -1, dh)[:, :L]    # [hkv, L, dh]
        V = kvf[pages, 1].transpose(1, 0, 2, 3).reshape(hkv, -1, dh)[:, :L]
        rows = int(k[b]) + 1
        ctx = L - rows
        Q = hid[r0:r0 + rows].reshape(rows, hq, dh)
        for h in range(hq):
            S = Q[:, h] @ K[h // g].T / math.sqrt(dh)                         # [rows, L]
            vis = np.arange(L)[None, :] < (ctx + np.arange(rows)[:, None] + 1)
            S = np.where(vis, S, -np.inf)
            P = np.exp(S - S.max(axis=1, keepdims=True))
            P /= P.sum(axis=1, keepdims=True)
            out[r0:r0 + rows, h * dh:(h + 1) * dh] = P @ V[h // g]
        r0 += rows
    return out


def test_attention_matches_dense_brute_force():
    rng = np.random.RandomState(2)
    hq, hkv, dh = 8, 2, 16
    case = _attn_case(rng, 3, hq, hkv, dh, [3, 0, 5], [37, 16, 1])
    got64, got16 = oracle.attention(*case[:3], case[3], case[4], hq, hkv, dh)
    want = _dense_attention(*case, hq, hkv, dh)
    assert np.max(np.abs(got64 - want)) < 1e-12
    assert np.array_equal(got16, oracle.f64_to_bf16(got64))


def test_attention_mha_matches_torch_sdpa_fp64():
    rng = np.random.RandomState(3)
    h, dh, k, ctx = 4, 32, 4, 45
    hidden, kv, pt, kv_len, kk = _attn_case(rng, 1, h, h, dh, [k], [ctx])
    got64, _ = oracle.attention(hidden, kv, pt, kv_len, kk, h, h, dh)
    L = int(kv_len[0])
    kvf = torch.from_numpy(oracle.bf16_to_f64(kv))
    pages = torch.from_numpy(pt[0, :(L + 15) // 16].astype(np.int64))
    K = kvf[pages, 0].permute(1, 0, 2, 3).reshape(h, -1, dh)[:, :L]
    V = kvf[pages, 1].permute(1, 0, 2, 3).reshape(h, -1, dh)[:, :L]
    Q = torch.from_numpy(oracle.bf16_to_f64(hidden)).reshape(k + 1, h, dh).permute(1, 0, 2)
    mask = torch.arange(L)[None, :] < (ctx + torch.arange(k + 1)[:, None] + 1)
    ref = torch.nn.functional.scaled_dot_product_attention(Q[None], K[None], V[None],
                                                           attn_mask=mask[None, None])
    ref = ref[0].permute(1, 0, 2).reshape(k + 1, h * dh).numpy()
    assert np.max(np.abs(got64 - ref)) < 1e-12


def test_attention_special_cases():
    rng = np.random.RandomState(4)
    hq, hkv, dh = 4, 2, 16
    # one visible token: row 0 with no committed context returns V[0]
    hidden, kv, pt, kv_len, k = _attn_case(rng, 1, hq, hkv, dh, [2], [0])
    got64, _ = oracle.attention(hidden, kv, pt, kv_len, k, hq, hkv, dh)
    kvf = oracle.bf16_to_f64(kv)
    for h in range(hq):
        assert np.array_equal(got64[0, h * dh:(h + 1) * dh], kvf[pt[0, 0], 1, h // 2, 0])
    # all keys equal: uniform attention, output = mean of the visible values
    hidden, kv, pt, kv_len, k = _attn_case(rng, 1, hq, hkv, dh, [3], [21])
    kv[:, 0] = kv[0, 0, 0, 0][None, None, None, :]
    got64, _ = oracle.attention(hidden, kv, pt, kv_len, k, hq, hkv, dh)
    kvf = oracle.bf16_to_f64(kv)
    L = int(kv_len[0])
    V = kvf[pt[0, :(L + 15) // 16], 1].transpose(1, 0, 2, 3).reshape(hkv, -1, dh)
    for j in range(4):
        n_vis = 21 + j + 1
        for h in range(hq):
            want = V[h // 2, :n_vis].mean(axis=0)
            assert np.max(np.abs(got64[j, h * dh:(h + 1) * dh] - want)) < 1e-13


def test_attention_invariants_causality_paging_selection():
    rng = np.random.RandomState(5)
    hq, hkv, dh = 8, 4, 16
    hidden, kv, pt, kv_len, k = _attn_case(rng, 2, hq, hkv, dh, [4, 2], [30, 19])
    base, _ = oracle.attention(hidden, kv, pt, kv_len, k, hq, hkv, dh)
    # causality inside the draft window: changing K/V at positions >= n_vis of row j leaves row j alone
    kv2 = kv.copy()
    j = 1
    first_hidden = 30 + j + 1
    for t in range(first_hidden, int(kv_len[0])):
        kv2[pt[0, t // 16], :, :, t % 16, :] = _rand_bf16(rng, (2, hkv, dh))
    pert, _ = oracle.attention(hidden, kv2, pt, kv_len, k, hq, hkv, dh)
    assert np.array_equal(pert[:j + 1], base[:j + 1])
    assert not np.array_equal(pert[j + 1:5], base[j + 1:5])
    assert np.array_equal(pert[5:], base[5:])
    # physical page permutation + matching table: unchanged
    perm = rng.permutation(kv.shape[0])
    inv = np.argsort(perm)
    kv3 = kv[perm]
    pt3 = np.where(pt >= 0, inv[np.maximum(pt, 0)], -1).astype(np.int32)
    moved, _ = oracle.attention(hidden, kv3, pt3, kv_len, k, hq, hkv, dh)
    assert np.array_equal(moved, base)
    # evaluating a subset of sequences gives the same rows
    sub, _ = oracle.attention(hidden, kv, pt, kv_len, k, hq, hkv, dh, seq_sel=[1])
    assert np.array_equal(sub[5:], base[5:]) and not sub[:5].any()


# --------------------------------------------------------------- LM head

def test_lm_head_matches_fp64_matmul():
    rng = np.random.RandomState(6)
    x = _rand_bf16(rng, (7, 96))
    w = _rand_bf16(rng, (301, 96))
    got = oracle.lm_head(x, w)
    want = oracle.bf16_to_f64(x) @ oracle.bf16_to_f64(w).T
    assert got.shape == (7, 301)
    assert np.max(np.abs(got - want)) < 1e-12 * np.max(np.abs(want))
    # not transposed: a non-square, asymmetric probe
    x1 = np.zeros((1, 96), np.uint16); x1[0, 5] = 0x3F80       # e_5
    assert np.array_equal(oracle.lm_head(x1, w)[0], oracle.bf16_to_f64(w)[:, 5])
    sub = oracle.lm_head(x, w, row_sel=[2, 6])
    assert np.array_equal(sub[[2, 6]], got[[2, 6]]) and not sub[[0, 1, 3, 4, 5]].any()


# --------------------------------------------------------------- softmax

def test_softmax_against_library_and_invariants():
    rng = np.random.RandomState(7)
    z = rng.standard_normal(1000) * 5
    for temp in (1.0, 0.7, 2.5):
        p = oracle.softmax(z, temp)
        assert abs(p.sum() - 1) < 1e-12
        assert np.max(np.abs(np.log(p) - scipy.special.log_softmax(z / temp))) < 1e-12
        assert np.max(np.abs(oracle.softmax(z + 123.0 * temp, temp) - p)) < 1e-13
    z[10] = -np.inf
    z[11] = 1e4                       # would overflow without max subtraction
    p = oracle.softmax(z, 1.0)
    assert p[10] == 0.0 and abs(p[11] - 1.0) < 1e-12 and np.isfinite(p).all()
    mask = np.full((1000 + 31) // 32, 0xFFFFFFFF, np.uint32)
    mask[0] &= ~np.uint32(1 << 3)     # forbid token 3
    mask[11 // 32] &= ~np.uint32(1 << 11)
    p = oracle.softmax(z, 1.0, mask)
    assert p[3] == 0.0 and p[11] == 0.0 and abs(p.sum() - 1) < 1e-12
    keep = np.ones(1000, bool); keep[[3, 10, 11]] = False
    assert np.max(np.abs(p[keep] - scipy.special.softmax(z[keep]))) < 1e-13


# ------------------------------------------------- acceptance + emission

def _logits_for(p):
    with np.errstate(divide="ignore"):
        return np.log(p)


def test_greedy_golden_cases():
    cases = []
    with open(os.path.join(GOLD, "greedy_cases.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            a, b, c, d = [t.strip() for t in line.split("|")]
            draft = [] if a == "-" else [int(t) for t in a.split(",")]
            cases.append((draft, [int(t) for t in b.split(",")], int(c), int(d)))
    assert len(cases) == 7
    rng = np.random.RandomState(8)
    v = 6
    # all cases in one ragged batch
    zt, toks, lens = [], [], []
    for draft, amax, _, _ in cases:
        for a in amax:
            row = rng.standard_normal(v)
            row[a] = row.max() + 1.0
            zt.append(row)
        toks += draft
        lens.append(len(draft))
    res = oracle.accept(oracle.GREEDY, np.array(zt), None, np.array(toks, np.int32),
                        np.array(lens, np.int32), np.zeros(len(cases), np.uint64))
    assert list(res["accepted_len"]) == [c[2] for c in cases]
    assert list(res["next_token"]) == [c[3] for c in cases]
    # ties: lowest index wins
    z = np.zeros((1, v)); z[0, [2, 4]] = 1.0
    res = oracle.accept(oracle.GREEDY, z, None, None, np.array([0], np.int32), np.zeros(1, np.uint64))
    assert res["next_token"][0] == 2


def test_sample_p_equals_q_accepts_everything():
    rng = np.random.RandomState(9)
    v, k, b = 50, 6, 200
    z = rng.standard_normal((b * (k + 1), v)).astype(np.float32) * 3
    zd = z.reshape(b, k + 1, v)[:, :k].reshape(b * k, v).copy()
    toks = rng.randint(0, v, b * k).astype(np.int32)
    res = oracle.accept(oracle.SAMPLE, z.astype(np.float64), zd, toks, np.full(b, k, np.int32),
                        rng.randint(0, 2 ** 62, b).astype(np.uint64), temperature=0.8)
    assert np.all(res["accepted_len"] == k)
    assert np.allclose(res["p_tok"], res["q_tok"], rtol=0, atol=0)


def _explicit_inverse_cdf(r, thr):
    c = np.cumsum(r)
    hit = np.nonzero(c > thr)[0]
    return int(hit[0]) if hit.size else int(np.nonzero(r > 0)[0][-1])


def test_sample_k0_is_plain_sampling_from_p():
    rng = np.random.RandomState(10)
    v, b = 13, 4000
    z = rng.standard_normal((b, v)) * 2
    seeds = rng.randint(0, 2 ** 62, b).astype(np.uint64)
    res = oracle.accept(oracle.SAMPLE, z, np.zeros((0, v), np.float32), None,
                        np.zeros(b, np.int32), seeds, temperature=1.3)
    assert np.all(res["accepted_len"] == 0)
    for i in range(b):
        p = scipy.special.softmax(z[i] / 1.3)
        u2 = oracle.uniform(int(seeds[i]), 0, 1)
        assert res["next_token"][i] == _explicit_inverse_cdf(p, u2 * p.sum())


def test_sample_rule_and_residual_brute_force():
    """Every decision recomputed from the definition with library softmax."""
    rng = np.random.RandomState(11)
    v, b = 9, 3000
    k = rng.randint(0, 5, b).astype(np.int32)
    m, s = int(k.sum()) + b, int(k.sum())
    zt = rng.standard_normal((m, v)) * 2
    zd = (rng.standard_normal((s, v)) * 2).astype(np.float32)
    zd[rng.rand(s, v) < 0.15] = -np.inf          # holes in the draft support
    zd[:, 0] = np.where(np.isinf(zd).all(axis=1), 0.0, zd[:, 0])
    toks = rng.randint(0, v, s).astype(np.int32)
    seeds = rng.randint(0, 2 ** 62, b).astype(np.uint64)
    temp = 0.9
    res = oracle.accept(oracle.SAMPLE, zt, zd, toks, k, seeds, temperature=temp)
    r0 = np.concatenate([[0], np.cumsum(k + 1)])
    t0 = np.concatenate([[0], np.cumsum(k)])
    n_resampled = 0
    for i in range(b):
        n = int(k[i])
        for j in range(int(k[i])):
            p = scipy.special.softmax(zt[r0[i] + j] / temp)
            q = scipy.special.softmax(zd[t0[i] + j].astype(np.float64) / temp)
            x = toks[t0[i] + j]
            u = oracle.uniform(int(seeds[i]), j, 0)
            assert abs(res["p_tok"][t0[i] + j] - p[x]) < 1e-14
            assert abs(res["q_tok"][t0[i] + j] - q[x]) < 1e-14
            ratio = 1.0 if q[x] <= p[x] else p[x] / q[x]
            if abs(u - ratio) > 1e-9:
                if not (u < ratio):
                    n = j
                    break
        assert res["accepted_len"][i] == n
        p = scipy.special.softmax(zt[r0[i] + n] / temp)
        if n < k[i]:
            q = scipy.special.softmax(zd[t0[i] + n].astype(np.float64) / temp)
            r = np.maximum(0.0, p - q)
            n_resampled += 1
            # residual mass identity: sum max(0,p-q) = 1 - sum min(p,q)
            assert abs(res["resid_mass"][i] - (1 - np.minimum(p, q).sum())) < 1e-12
        else:
            r = p
        u2 = oracle.uniform(int(seeds[i]), n, 1)
        if res["cdf_margin"][i] > 1e-9:
            assert res["next_token"][i] == _explicit_inverse_cdf(r, u2 * r.sum())
    assert n_resampled > 500


def test_sample_zero_probability_conventions():
    v = 4
    # draft proposes a token the target forbids: rejected for every u; the residual is p
    zt = _logits_for(np.array([[0.0, 0.5, 0.5, 0.0], [0.25, 0.25, 0.25, 0.25]]))
    zd = _logits_for(np.array([[1.0, 0.0, 0.0, 0.0]])).astype(np.float32)
    for seed in range(200):
        res = oracle.accept(oracle.SAMPLE, zt, zd, np.array([0], np.int32), np.array([1], np.int32),
                            np.array([seed], np.uint64))
        assert res["accepted_len"][0] == 0 and res["next_token"][0] in (1, 2)
        assert abs(res["resid_mass"][0] - 1.0) < 1e-15
    # the same through a vocabulary mask on finite target logits
    zt2 = np.zeros((2, v))
    mask = np.array([[0b0110]], np.uint32)
    for seed in range(200):
        res = oracle.accept(oracle.SAMPLE, zt2, zd, np.array([0], np.int32), np.array([1], np.int32),
                            np.array([seed], np.uint64), vocab_mask=mask)
        assert res["accepted_len"][0] == 0 and res["next_token"][0] in (1, 2)
    # q(x) = 0 < p(x): always accepted
    zd3 = _logits_for(np.array([[0.0, 1.0, 0.0, 0.0]])).astype(np.float32)
    for seed in range(50):
        res = oracle.accept(oracle.SAMPLE, zt, zd3, np.array([2], np.int32), np.array([1], np.int32),
                            np.array([seed], np.uint64))
        assert res["accepted_len"][0] == 1


def test_sample_low_temperature_limit_is_greedy():
    rng = np.random.RandomState(12)
    v, b, k = 11, 300, 4
    zt = rng.standard_normal((b * (k + 1), v))
    zt[np.arange(zt.shape[0]), zt.argmax(-1)] += 5.0        # a clear winner in every row
    toks = np.where(rng.rand(b * k) < 0.7,
                    zt.reshape(b, k + 1, v)[:, :k].argmax(-1).reshape(-1),
                    rng.randint(0, v, b * k)).astype(np.int32)
    zd = np.full((b * k, v), -np.inf, np.float32)
    zd[np.arange(b * k), toks] = 0.0                       # one-hot draft
    lens = np.full(b, k, np.int32)
    seeds = rng.randint(0, 2 ** 62, b).astype(np.uint64)
    g = oracle.accept(oracle.GREEDY, zt, None, toks, lens, seeds)
    s = oracle.accept(oracle.SAMPLE, zt, zd, toks, lens, seeds, temperature=1e-3)
    assert np.array_equal(g["accepted_len"], s["accepted_len"])
    assert np.array_equal(g["next_token"], s["next_token"])


def _trial_batch(p_rows, q_rows, n, rng, k):
    """n independent sequences sharing the same rows; x_j ~ q_j drawn by the harness."""
    v = p_rows.shape[1]
    zt = np.tile(_logits_for(p_rows), (n, 1))
    zd = np.tile(_logits_for(q_rows).astype(np.float32), (n, 1))
    toks = np.stack([rng.choice(v, size=n, p=q_rows[j]) for j in range(k)], axis=1).astype(np.int32)
    seeds = rng.randint(0, 2 ** 62, n).astype(np.uint64)
    res = oracle.accept(oracle.SAMPLE, zt, zd, toks.reshape(-1), np.full(n, k, np.int32), seeds)
    return toks, res


def test_lossless_chi_square_million_trials():
    """The first emitted token (accepted x_0, or the resample) follows p_0; given x_0 accepted
    the second emitted token follows p_1 -- chi-square at the 99.9% level, 10^6 seeded trials."""
    rng = np.random.RandomState(13)
    v, k, n = 12, 2, 1_000_000
    p_rows = rng.dirichlet(np.ones(v) * 0.7, size=k + 1)
    q_rows = rng.dirichlet(np.ones(v) * 0.7, size=k)
    q_rows[0, 3] = 0.0; q_rows[0] /= q_rows[0].sum()       # a hole in the draft's support
    # fp32 draft logits: the q the oracle sees
    q_seen = np.stack([scipy.special.softmax(_logits_for(q_rows[j]).astype(np.float32).astype(np.float64))
                       for j in range(k)])
    counts0 = np.zeros(v)
    counts1 = np.zeros(v)
    n_acc0 = 0
    acc_rate = 0.0
    for chunk in range(10):
        toks, res = _trial_batch(p_rows, q_rows, n // 10, rng, k)
        a = res["accepted_len"]
        first = np.where(a >= 1, toks[:, 0], res["next_token"])
        counts0 += np.bincount(first, minlength=v)
        got0 = a >= 1
        second = np.where(a >= 2, toks[:, 1], res["next_token"])[got0]
        counts1 += np.bincount(second, minlength=v)
        n_acc0 += int(got0.sum())
        acc_rate += float(got0.mean()) / 10
    chi0 = ((counts0 - n * p_rows[0]) ** 2 / (n * p_rows[0])).sum()
    chi1 = ((counts1 - n_acc0 * p_rows[1]) ** 2 / (n_acc0 * p_rows[1])).sum()
    bound = scipy.stats.chi2.ppf(0.999, v - 1)
    assert chi0 < bound, (chi0, bound)
    assert chi1 < bound, (chi1, bound)
    # closed form: P(accept at 0) = sum_v min(p_0, q_0) = 1 - TV(p_0, q_0)
    want = np.minimum(p_rows[0], q_seen[0]).sum()
    assert abs(acc_rate - want) < 5 * math.sqrt(want * (1 - want) / n)


def test_flat_target_acceptance_closed_form():
    """Flat target and q ~ softmax(sigma * g): E[accept] = 2 * Phi(-sigma / (2 T))."""
    rng = np.random.RandomState(14)
    v, n = 4096, 400
    for sigma, temp in [(0.77, 1.0), (0.5, 1.0), (1.5, 1.0), (0.77 * 0.7, 0.7)]:
        zd = (rng.standard_normal((n, v)) * sigma).astype(np.float32)
        zt = np.zeros((2 * n, v))
        q = scipy.special.softmax(zd.astype(np.float64) / temp, axis=1)
        toks = np.array([rng.choice(v, p=q[i]) for i in range(n)], np.int32)
        res = oracle.accept(oracle.SAMPLE, zt, zd, toks, np.ones(n, np.int32),
                            rng.randint(0, 2 ** 62, n).astype(np.uint64), temperature=temp)
        want = 2 * scipy.stats.norm.cdf(-sigma / (2 * temp))
        exact = np.minimum(q, 1.0 / v).sum(axis=1).mean()
        assert abs(exact - want) < 0.01
        assert abs(res["accepted_len"].mean() - exact) < 4 * math.sqrt(0.25 / n)


def test_whole_step_composition_and_rollback_contract():
    """verify() = attention -> bf16 -> LM head -> accept; accepted_len is in [0,k] and the
    emitted block has accepted_len+1 tokens (Algorithm 2: draft[1:tau] followed by x_new)."""
    rng = np.random.RandomState(15)
    hq, hkv, dh, v = 4, 2, 16, 64
    hidden, kv, pt, kv_len, k = _attn_case(rng, 3, hq, hkv, dh, [3, 0, 2], [20, 9, 33])
    w = _rand_bf16(rng, (v, hq * dh))
    s = int(k.sum())
    zd = rng.standard_normal((s, v)).astype(np.float32)
    toks = rng.randint(0, v, s).astype(np.int32)
    seeds = np.array([5, 6, 7], np.uint64)
    res = oracle.verify(oracle.SAMPLE, hidden, kv, pt, kv_len, k, w, toks, zd, seeds, hq, hkv, dh)
    assert np.array_equal(res["attn_bf16"], oracle.f64_to_bf16(res["attn_f64"]))
    want_logits = oracle.bf16_to_f64(res["attn_bf16"]) @ oracle.bf16_to_f64(w).T
    assert np.max(np.abs(res["logits"] - want_logits)) < 1e-12
    assert np.all((res["accepted_len"] >= 0) & (res["accepted_len"] <= k))
    assert np.all((res["next_token"] >= 0) & (res["next_token"] < v))
    sub = oracle.verify(oracle.SAMPLE, hidden, kv, pt, kv_len, k, w, toks, zd, seeds, hq, hkv, dh,
                        seq_sel=[2])
    assert sub["accepted_len"][2] == res["accepted_len"][2]
    assert sub["next_token"][2] == res["next_token"][2]
    assert sub["accepted_len"][0] == -1


# ------------------------------------------------------------- KV session

def test_kv_append_and_rollback_against_direct_indexing():
    """Section IV-C: the window's K/V rows land at positions ctx .. ctx+k of the sequence (checked by
    reading them back through the page table with plain numpy indexing, and by the fact that attention
    over the appended pool equals attention over a pool that held those rows all along); the rollback
    keeps context + accepted drafts + the window's first position."""
    rng = np.random.RandomState(21)
    hq, hkv, dh = 4, 2, 16
    k = np.array([3, 0, 5], np.int32)
    ctx = np.array([20, 9, 33], np.int32)
    hidden, kv, pt, kv_len, k2 = _attn_case(rng, 3, hq, hkv, dh, list(k), list(ctx))
    assert np.array_equal(k, k2)
    m = int(k.sum()) + 3
    new_k = rng.randint(0, 2 ** 15, (m, hkv, dh)).astype(np.uint16)
    new_v = rng.randint(0, 2 ** 15, (m, hkv, dh)).astype(np.uint16)
    pool = oracle.kv_append(kv, pt, kv_len, k, new_k, new_v, hkv, dh)
    touched = np.zeros(kv.shape, bool)
    row = 0
    for b in range(3):
        for j in range(k[b] + 1):
            t = kv_len[b] - (k[b] + 1) + j
            page, slot = pt[b, t // 16], t % 16
            assert np.array_equal(pool[page, 0, :, slot, :], new_k[row])
            assert np.array_equal(pool[page, 1, :, slot, :], new_v[row])
            touched[page, :, :, slot, :] = True
            row += 1
    assert np.array_equal(pool[~touched], kv[~touched])            # nothing else was written
    # attention sees exactly the appended rows
    a_new, _ = oracle.attention(hidden, pool, pt, kv_len, k, hq, hkv, dh)
    a_old, _ = oracle.attention(hidden, kv, pt, kv_len, k, hq, hkv, dh)
    assert not np.allclose(a_new, a_old)
    # rollback: all accepted keeps everything but the bonus position's successor; none accepted keeps ctx + 1
    acc = np.array([3, 0, 2], np.int32)
    nxt = oracle.kv_rollback(kv_len, k, acc)
    assert list(nxt) == [20 + 3 + 1, 9 + 0 + 1, 33 + 2 + 1]
    assert np.all(nxt <= kv_len) and np.all(nxt >= kv_len - k)


# ------------------------------------------------------------------ top-p

def test_nucleus_against_numpy_sort_and_its_invariants():
    rng = np.random.RandomState(31)
    for v, top_p in [(7, 0.5), (50, 0.9), (1000, 0.9), (1000, 0.3), (64, 0.999)]:
        p = rng.dirichlet(np.ones(v) * 0.3)
        got, margin = oracle.nucleus(p, top_p)
        order = np.lexsort((np.arange(v), -p))                    # decreasing p, ties by index
        c = np.cumsum(p[order])
        m = int(np.searchsorted(c, top_p, side="left"))           # first prefix with mass >= top_p
        keep = p >= p[order[m]]
        want = np.where(keep, p, 0.0) / p[keep].sum()
        assert np.allclose(got, want, rtol=0, atol=1e-15)
        assert abs(got.sum() - 1) < 1e-12
        assert p[keep].sum() >= top_p and (m == 0 or c[m - 1] < top_p)   # minimal prefix
        assert np.isclose(margin, min(abs(c[m] - top_p), abs(top_p - (c[m - 1] if m else 0.0))))
    # ties with the last kept token are all kept; top_p >= 1 is the identity
    p = np.array([0.4, 0.2, 0.2, 0.2])
    got, _ = oracle.nucleus(p, 0.5)
    assert np.allclose(got, [0.4, 0.2, 0.2, 0.2])
    got, _ = oracle.nucleus(p, 0.3)
    assert np.allclose(got, [1, 0, 0, 0])
    got, m = oracle.nucleus(p, 1.0)
    assert np.array_equal(got, p) and m == np.inf


def test_top_p_sampling_is_lossless_with_respect_to_the_nucleus():
    """With top_p < 1 the emitted token follows the nucleus of the target row (chi-square, 4*10^5
    trials), a draft token outside the nucleus is always rejected, and top_p = 1 changes nothing."""
    rng = np.random.RandomState(32)
    v, n = 12, 400_000
    p0 = rng.dirichlet(np.ones(v) * 0.7)
    p1 = rng.dirichlet(np.ones(v) * 0.7)
    q0 = rng.dirichlet(np.ones(v) * 0.7)
    top_p = 0.8
    zt = np.tile(np.stack([_logits_for(p0), _logits_for(p1)]), (n, 1))
    zd32 = _logits_for(q0).astype(np.float32)
    q_seen = scipy.special.softmax(zd32.astype(np.float64))
    zd = np.tile(zd32[None, :], (n, 1))
    toks = rng.choice(v, size=n, p=q_seen).astype(np.int32)
    seeds = rng.randint(0, 2 ** 62, n).astype(np.uint64)
    res = oracle.accept(oracle.SAMPLE, zt, zd, toks, np.ones(n, np.int32), seeds, top_p=top_p)
    nuc0, _ = oracle.nucleus(p0, top_p)
    first = np.where(res["accepted_len"] >= 1, toks, res["next_token"])
    counts = np.bincount(first, minlength=v).astype(np.float64)
    assert np.all(counts[nuc0 == 0] == 0)                          # nothing outside the nucleus is ever emitted
    sup = nuc0 > 0
    chi = ((counts[sup] - n * nuc0[sup]) ** 2 / (n * nuc0[sup])).sum()
    assert chi < scipy.stats.chi2.ppf(0.999, int(sup.sum()) - 1), chi
    outside = (nuc0[toks] == 0)
    assert outside.any() and np.all(res["accepted_len"][outside] == 0)
    assert np.allclose(res["p_tok"], nuc0[toks])
    same = oracle.accept(oracle.SAMPLE, zt[:2000], zd[:1000], toks[:1000], np.ones(1000, np.int32), seeds[:1000], top_p=1.0)
    base = oracle.accept(oracle.SAMPLE, zt[:2000], zd[:1000], toks[:1000], np.ones(1000, np.int32), seeds[:1000])
    assert np.array_equal(same["next_token"], base["next_token"]) and np.array_equal(same["accepted_len"], base["accepted_len"])


# ------------------------------------------------------------------ top-k, per-sequence temperature, page release

def test_top_k_filter_against_a_numpy_sort():
    rng = np.random.RandomState(41)
    for v, k in [(7, 3), (50, 1), (1000, 40), (1000, 999), (64, 64), (64, 0), (64, 200)]:
        p = rng.dirichlet(np.full(v, 0.3))
        got = oracle.topk(p, k)
        if k <= 0 or k >= v:
            assert np.array_equal(got, p)
            continue
        order = np.lexsort((np.arange(v), -p))
        keep = order[:k]
        want = np.zeros(v)
        want[keep] = p[keep] / p[keep].sum()
        assert np.allclose(got, want, rtol=0, atol=1e-15)
        assert np.count_nonzero(got) == k and abs(got.sum() - 1.0) < 1e-12
    # ties with the k-th token are all kept
    p = np.array([0.3, 0.2, 0.2, 0.2, 0.1])
    assert np.count_nonzero(oracle.topk(p, 2)) == 4
    assert np.count_nonzero(oracle.topk(p, 1)) == 1
    # top-k comes before top-p: the nucleus is taken of the renormalised top-k distribution
    p = np.array([0.4, 0.3, 0.2, 0.1])
    both, _ = oracle.nucleus(oracle.topk(p, 2), 0.6)           # top-2 -> (4/7, 3/7); mass 0.6 needs both
    assert np.allclose(both, [4 / 7, 3 / 7, 0, 0])
    r, z = oracle.emission(np.log(p), None, top_k=2, top_p=0.6)
    assert np.allclose(r, both) and abs(z - 1.0) < 1e-12


def test_top_k_sampling_follows_the_filtered_target():
    """With top_k the emitted token follows the top-k filtered target row (chi-square over 3*10^5
    trials) and a draft token outside the top-k set is always rejected."""
    rng = np.random.RandomState(43)
    v, n, top_k = 12, 300000, 5
    z_t = rng.standard_normal(v) * 1.5
    z_d = (z_t + rng.standard_normal(v)).astype(np.float32)
    p0 = np.exp(z_t - z_t.max()); p0 /= p0.sum()
    pk = oracle.topk(p0, top_k)
    q0 = np.exp(z_d.astype(np.float64) - z_d.max()); q0 /= q0.sum()
    toks = rng.choice(v, size=n, p=q0).astype(np.int32)
    zt = np.tile(z_t, (2 * n, 1))
    zd = np.tile(z_d, (n, 1))
    seeds = rng.randint(0, 2 ** 62, n).astype(np.uint64)
    res = oracle.accept(oracle.SAMPLE, zt, zd, toks, np.ones(n, np.int32), seeds, top_k=top_k)
    outside = pk[toks] == 0.0
    assert outside.any() and np.all(res["accepted_len"][outside] == 0)
    first = np.where(res["accepted_len"] >= 1, toks, res["next_token"])
    counts = np.bincount(first, minlength=v).astype(np.float64)
    assert np.all(counts[pk == 0.0] == 0)
    sup = pk > 0
    chi2 = float((((counts[sup] - n * pk[sup]) ** 2) / (n * pk[sup])).sum())
    assert chi2 < scipy.stats.chi2.ppf(0.999, sup.sum() - 1)


def test_per_sequence_temperatures_equal_separate_runs():
    rng = np.random.RandomState(47)
    v, batch = 300, 6
    k = rng.randint(0, 5, batch).astype(np.int32)
    m, s = int(k.sum()) + batch, int(k.sum())
    zt = rng.standard_normal((m, v)) * 2
    zd = (rng.standard_normal((s, v)) * 2).astype(np.float32)
    toks = rng.randint(0, v, s).astype(np.int32)
    seeds = rng.randint(0, 2 ** 62, batch).astype(np.uint64)
    temps = np.array([0.5, 1.0, 0.7, 1.3, 2.0, 0.9])
    res = oracle.accept(oracle.SAMPLE, zt, zd, toks, k, seeds, temperature=123.0, temperatures=temps)
    for b in range(batch):
        one = oracle.accept(oracle.SAMPLE, zt, zd, toks, k, seeds, temperature=float(temps[b]), seq_sel=[b])
        assert one["accepted_len"][b] == res["accepted_len"][b] and one["next_token"][b] == res["next_token"][b]
    t0 = np.concatenate([[0], np.cumsum(k)])
    r0 = np.concatenate([[0], np.cumsum(k + 1)])
    for b in range(batch):                       # p(x_j) against scipy at the sequence's own temperature
        for j in range(k[b]):
            want = scipy.special.softmax(zt[r0[b] + j] / temps[b])[toks[t0[b] + j]]
            assert abs(res["p_tok"][t0[b] + j] - want) < 1e-14


def test_kv_release_returns_exactly_the_pages_past_the_new_length():
    rng = np.random.RandomState(53)
    batch, max_pages = 5, 12
    prev = np.array([100, 33, 16, 48, 17], np.int32)           # lengths before the rollback
    nxt = np.array([96, 33, 1, 31, 16], np.int32)              # after: pages kept = ceil(next / 16)
    pt = np.full((batch, max_pages), -1, np.int32)
    ids = rng.permutation(200).astype(np.int32)
    c = 0
    for b in range(batch):
        n = -(-int(prev[b]) // 16)
        pt[b, :n] = ids[c:c + n]; c += n
    new_pt, freed = oracle.kv_release(pt, prev, nxt)
    want = []
    for b in range(batch):
        keep, had = -(-int(nxt[b]) // 16), -(-int(prev[b]) // 16)
        want += list(pt[b, keep:had])
        assert np.array_equal(new_pt[b, :keep], pt[b, :keep]) and np.all(new_pt[b, keep:] == -1)
    assert list(freed) == want and len(freed) == (7 - 6) + 0 + 0 + (3 - 2) + (2 - 1)
    # nothing to release when nothing was rejected
    same_pt, none = oracle.kv_release(pt, prev, prev)
    assert np.array_equal(same_pt, pt) and len(none) == 0
