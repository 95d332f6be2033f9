"""Shared helpers of the GPU parity tests: run the CUDA path through the C ABI binding and the
fp64 oracle on the same seeded inputs, and compare stage by stage.

Draft logits of the sequences that are compared are  oracle target logits + noise  (the
configs' "draft = target + N(0, sigma)" model); the other sequences of a full-size batch get the
noise alone -- with N(0, 0.02) inputs the target logits are ~5e-4, far below the noise, so the
acceptance statistics are unchanged.  Nothing the oracle consumes comes from the CUDA path.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2601_00644_b200 import workloads as wl

REL_TOL = 2e-2        # attention outputs and logits: bf16 inputs, fp32 accumulation
PROB_TOL = 1e-5       # probabilities, absolute
TIE_TOL = 1e-5        # |u - min(1, p/q)| below this is a near-tie: counted, not required to match
CDF_TIE_TOL = 1e-6    # inverse-CDF boundary: fp32 exponentials (2^-22 rel.) against fp64


def rel_close(got: np.ndarray, ref: np.ndarray, tol: float = REL_TOL):
    """Row-wise max|d|/max|ref| and element-wise |d| <= tol*|ref| + tol*rms(ref)."""
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    d = np.abs(got - ref)
    row_scale = np.maximum(np.abs(ref).max(axis=-1, keepdims=True), 1e-300)
    row_err = float((d.max(axis=-1, keepdims=True) / row_scale).max())
    rms = np.sqrt((ref ** 2).mean(axis=-1, keepdims=True))
    elem_ok = bool(np.all(d <= tol * np.abs(ref) + tol * rms))
    return row_err, elem_ok


class Case:
    """One verification workload on the GPU plus its host copies for the oracle."""

    def __init__(self, shape: wl.VerifyShape, check_seqs=None, device="cuda", mode=0,
                 vocab_mask=None):
        self.shape = shape
        self.inp = wl.make_inputs(shape, device=device)
        inp = self.inp
        self.batch = inp.batch
        self.k = inp.draft_len.cpu().numpy()
        self.kv_len = inp.kv_len.cpu().numpy()
        self.row0 = inp.row_offsets()
        self.tok0 = inp.tok_offsets()
        self.check = list(range(self.batch)) if check_seqs is None else list(check_seqs)
        self.mode = mode
        # host copies for the oracle
        self.h_hidden = wl.bits_u16(inp.hidden)
        self.h_kv = wl.bits_u16(inp.kv_pages)
        self.h_pt = inp.page_table.cpu().numpy()
        self.h_w = wl.bits_u16(inp.lm_head_w)
        self.h_seeds = wl.seeds_u64(inp.seeds)
        self.vocab_mask = vocab_mask                      # numpy uint32 [B, words] or None
        self._oracle_front = None

    # ---- oracle: attention + LM head on the checked sequences
    def oracle_front(self):
        if self._oracle_front is None:
            s = self.shape
            a64, a16 = oracle.attention(self.h_hidden, self.h_kv, self.h_pt, self.kv_len, self.k,
                                        s.n_q_heads, s.n_kv_heads, s.head_dim, 16, self.check)
            rows = self.rows_of(self.check)
            logits = oracle.lm_head(a16, self.h_w, rows)
            self._oracle_front = (a64, a16, logits)
        return self._oracle_front

    def rows_of(self, seqs):
        return np.concatenate([np.arange(self.row0[b], self.row0[b + 1]) for b in seqs]).astype(np.int32)

    def drows_of(self, seqs):
        parts = [np.arange(self.tok0[b], self.tok0[b + 1]) for b in seqs]
        return np.concatenate(parts).astype(np.int64) if parts else np.zeros(0, np.int64)

    # ---- draft logits / tokens
    def build_drafts(self):
        """draft logits = oracle target logits (rows j < k_b of the checked sequences) + noise."""
        inp = self.inp
        _, _, logits = self.oracle_front()
        dl = inp.noise.clone()
        for b in self.check:
            kb = int(self.k[b])
            if kb == 0:
                continue
            tgt = torch.from_numpy(logits[self.row0[b]:self.row0[b] + kb]).to(dl.device)
            dl[self.tok0[b]:self.tok0[b] + kb] = (tgt + dl[self.tok0[b]:self.tok0[b] + kb].double()).float()
        self.draft_logits = dl
        self.draft_tokens = wl.draw_draft_tokens(dl, self.shape.temperature, inp.token_uniforms)
        return dl, self.draft_tokens

    # ---- oracle: the decision stage
    def oracle_accept(self, target_logits_f64, draft_logits=None, draft_tokens=None, temperature=None, top_p=1.0,
                      top_k=0, temperatures=None):
        dl = self.draft_logits if draft_logits is None else draft_logits
        dt = self.draft_tokens if draft_tokens is None else draft_tokens
        t = self.shape.temperature if temperature is None else temperature
        return oracle.accept(self.mode, target_logits_f64,
                             None if dl is None else dl.cpu().numpy(), dt.cpu().numpy(), self.k,
                             self.h_seeds, t, self.vocab_mask, self.check, top_p=top_p, top_k=top_k,
                             temperatures=temperatures)


def make_verifier(case: Case, debug=True, mode=None):
    from paper_2601_00644_b200 import binding
    s = case.shape
    k_max = max(int(case.k.max()), 1)
    return binding.Verifier(case.inp.lm_head_w, s.n_q_heads, s.n_kv_heads, s.head_dim,
                            max_batch=case.batch, k_max=k_max,
                            max_kv_len=max(int(case.kv_len.max()), k_max + 1), mode=case.mode if mode is None else mode,
                            debug=debug)


CANARY = -0x5A5A5A5B          # guard-band pattern around output buffers
GUARD = 64                    # elements on either side


def guarded(n, dtype, device="cuda"):
    """A buffer of n elements with GUARD canary elements before and after it; returns (whole, view)."""
    per = torch.empty(0, dtype=dtype).element_size()
    words = ((n + 2 * GUARD) * per + 3) // 4
    raw = torch.full((words,), CANARY, dtype=torch.int32, device=device)
    whole = raw.view(dtype)
    return whole, whole[GUARD:GUARD + n]


def guards_intact(whole, n):
    raw = whole.view(torch.int32) if whole.dtype != torch.int32 else whole
    per = whole.element_size()
    lo = GUARD * per // 4
    hi = (GUARD + n) * per // 4 + (1 if ((GUARD + n) * per) % 4 else 0)
    return bool((raw[:lo] == CANARY).all() and (raw[hi:] == CANARY).all())


def run_gpu_verify(case: Case, ver, vocab_mask_dev=None, temperature=None):
    """One verify call; the two output arrays sit between canary guard bands that must survive it."""
    inp = case.inp
    t = case.shape.temperature if temperature is None else temperature
    acc_w, acc = guarded(case.batch, torch.int32)
    nxt_w, nxt = guarded(case.batch, torch.int32)
    ver.verify(inp.kv_pages, inp.page_table, inp.kv_len, inp.kv_len.cpu(), inp.hidden,
               case.draft_tokens, case.draft_logits, inp.draft_len, inp.draft_len.cpu(),
               inp.seeds, temperature=t, vocab_mask=vocab_mask_dev, accepted_len=acc, next_token=nxt)
    torch.cuda.synchronize()
    code, st = ver.status()
    assert code == 0, f"device status {code} {st}"
    assert guards_intact(acc_w, case.batch) and guards_intact(nxt_w, case.batch), "a kernel wrote outside accepted_len / next_token"
    return acc.cpu().numpy(), nxt.cpu().numpy()


def compare_decisions(case: Case, acc_gpu, nxt_gpu, ref, cdf_tol, label=""):
    """accepted_len / next_token against an oracle result `ref` computed from the SAME logits the
    GPU decided on.  Only genuine near-ties may differ: |u - min(1, p/q)| < TIE_TOL for an
    acceptance test, a CDF margin below `cdf_tol` for the emitted token.
    Returns (#accept near-ties, #cdf near-ties) that were excused."""
    ties = cdf_ties = 0
    for b in case.check:
        n_g, n_o = int(acc_gpu[b]), int(ref["accepted_len"][b])
        assert 0 <= n_g <= case.k[b]
        assert 0 <= nxt_gpu[b] < case.shape.vocab
        if n_g != n_o:
            j = min(n_g, n_o)
            margin = ref["acc_margin"][case.tok0[b] + j]
            assert margin < TIE_TOL, f"{label} seq {b}: accepted_len {n_g} vs oracle {n_o}, margin {margin}"
            ties += 1
            continue
        if int(nxt_gpu[b]) != int(ref["next_token"][b]):
            margin = ref["cdf_margin"][b]
            assert margin < cdf_tol, f"{label} seq {b}: next_token {nxt_gpu[b]} vs {ref['next_token'][b]}, cdf margin {margin}"
            cdf_ties += 1
    return ties, cdf_ties


def _ratio(p, q):
    """min(1, p/q) with the conventions of the acceptance test u*q < p (q = 0 < p accepts, p = 0 rejects)."""
    if p >= q:
        return 1.0 if p > 0.0 else 0.0
    return p / q


def compare_end_to_end(case: Case, acc_gpu, nxt_gpu, ref_own, ref_gpu_logits, logits_o, logits_g,
                       temperature, top_p=1.0, cdf_tol=CDF_TIE_TOL, label="end-to-end", top_k=0, temperatures=None):
    """GPU decisions against the oracle's own chain (its attention -> bf16 -> its LM head -> its decisions).

    The two sides decide on slightly different logits (a bf16 rounding of the attention output that
    falls the other way, fp32 accumulation order), and decisions are discontinuous in the logits.  A
    difference is accepted only in two cases, both evaluated by the oracle in fp64:
      near-tie    the oracle's own margin is below the near-tie tolerance (1e-5 for an acceptance
                  test, `cdf_tol` for the inverse-CDF boundary);
      explained   the oracle, fed the GPU's logits (`ref_gpu_logits`), takes the GPU's decision, and its
                  margin on its own logits is no larger than the distance the logit difference moves
                  the quantity that is compared:  |u - r_o| <= |r_g - r_o| for an acceptance test
                  (r = min(1, p/q) under the oracle's / the GPU's logits); for the emitted token
                  margin * Z_o <= max_v |C_g(v) - C_o(v)| + u' |Z_g - Z_o|  with C the running sums of
                  the emission weights in vocabulary order and Z their totals.
    Returns a dict of counts; anything else fails."""
    out = {"ties": 0, "cdf_ties": 0, "explained_accept": 0, "explained_token": 0}
    for b in case.check:
        n_g, n_o = int(acc_gpu[b]), int(ref_own["accepted_len"][b])
        t0 = case.tok0[b]
        if case.mode == 1:
            # greedy: every decision is an arg-max of one row.  At the first row where the two sides
            # disagree the two arg-max candidates must be closer in the oracle's logits than twice the
            # distance between the two logit sets, and the oracle on the GPU's logits must side with the GPU.
            if n_g == n_o and int(nxt_gpu[b]) == int(ref_own["next_token"][b]):
                continue
            row = case.row0[b] + min(n_g, n_o)
            zo, zg = logits_o[row], logits_g[row].astype(np.float64)
            gap = float(zo.max() - zo[int(np.argmax(zg))])
            shift = 2.0 * float(np.abs(zg - zo).max())
            assert (int(ref_gpu_logits["accepted_len"][b]) == n_g and int(ref_gpu_logits["next_token"][b]) == int(nxt_gpu[b])
                    and gap <= shift), f"{label} seq {b}: greedy ({n_g}, {nxt_gpu[b]}) vs ({n_o}, {ref_own['next_token'][b]}): gap {gap:.3e} > shift {shift:.3e}"
            out["explained_accept" if n_g != n_o else "explained_token"] += 1
            continue
        if n_g != n_o:
            j = t0 + min(n_g, n_o)
            margin = float(ref_own["acc_margin"][j])
            if margin < TIE_TOL:
                out["ties"] += 1
                continue
            r_o = _ratio(float(ref_own["p_tok"][j]), float(ref_own["q_tok"][j]))
            r_g = _ratio(float(ref_gpu_logits["p_tok"][j]), float(ref_gpu_logits["q_tok"][j]))
            assert int(ref_gpu_logits["accepted_len"][b]) == n_g and margin <= abs(r_g - r_o) + 1e-12, (
                f"{label} seq {b}: accepted_len {n_g} vs oracle {n_o}: margin {margin:.3e} is not covered by the "
                f"shift of min(1,p/q) between the two logit sets, {abs(r_g - r_o):.3e}")
            out["explained_accept"] += 1
            continue
        if int(nxt_gpu[b]) == int(ref_own["next_token"][b]):
            continue
        margin = float(ref_own["cdf_margin"][b])
        if margin < cdf_tol:
            out["cdf_ties"] += 1
            continue
        row = case.row0[b] + n_o
        drow = case.draft_logits[t0 + n_o].cpu().numpy() if n_o < case.k[b] else None
        mask = None if case.vocab_mask is None else case.vocab_mask[b]
        t_b = temperature if temperatures is None else float(temperatures[b])
        w_o, z_o = oracle.emission(logits_o[row], drow, t_b, top_p, mask, top_k=top_k)
        w_g, z_g = oracle.emission(logits_g[row].astype(np.float64), drow, t_b, top_p, mask, top_k=top_k)
        u2 = oracle.uniform(int(case.h_seeds[b]), n_o, 1)
        shift = float(np.abs(np.cumsum(w_g) - np.cumsum(w_o)).max()) + u2 * abs(z_g - z_o)
        assert int(ref_gpu_logits["next_token"][b]) == int(nxt_gpu[b]) and margin * z_o <= shift + 1e-15, (
            f"{label} seq {b}: next_token {nxt_gpu[b]} vs {ref_own['next_token'][b]}: cdf margin {margin * z_o:.3e} "
            f"is not covered by the shift of the running sums between the two logit sets, {shift:.3e}")
        out["explained_token"] += 1
    return out


def full_parity(case: Case, ver, vocab_mask_dev=None, top_p=1.0, top_k=0, temperatures=None):
    """Stage-by-stage and end-to-end comparison of one verify call.  Returns a report dict."""
    acc, nxt = run_gpu_verify(case, ver, vocab_mask_dev)
    m, s = case.inp.m_rows, case.inp.s_rows
    dbg = ver.debug(m, s)
    a64, a16, logits_o = case.oracle_front()
    rows = case.rows_of(case.check)
    drows = case.drows_of(case.check)
    t = case.shape.temperature
    rep = {}

    attn_g = dbg["attn_out"].float().cpu().numpy()
    rep["attn_row_err"], ok = rel_close(attn_g[rows], a64[rows])
    assert ok and rep["attn_row_err"] < REL_TOL, f"attention: {rep}"

    logits_g = dbg["logits"].cpu().numpy()
    rep["logit_row_err"], ok = rel_close(logits_g[rows], logits_o[rows])
    assert ok and rep["logit_row_err"] < REL_TOL, f"logits: {rep}"

    # (i) decision stage in isolation: the oracle is fed the GPU's own fp32 logits
    ref_iso = case.oracle_accept(logits_g.astype(np.float64), top_p=top_p, top_k=top_k, temperatures=temperatures)
    if top_p < 1.0:
        # a nucleus cut within 1e-6 of top_p is a near-tie of the filter itself: such sequences are
        # counted and left out of the identity requirement
        near = [b for b in case.check if ref_iso["topp_margin"][case.row0[b]:case.row0[b + 1]].min() < CDF_TIE_TOL]
        rep["topp_ties"] = len(near)
        case.check = [b for b in case.check if b not in near]
        drows = case.drows_of(case.check)
    if case.mode == 0:
        p_g = dbg["p_tok"].cpu().numpy()
        q_g = dbg["q_tok"].cpu().numpy()
        u_g = dbg["u"].cpu().numpy().astype(np.float64)
        if drows.size:
            rep["p_err"] = float(np.abs(p_g[drows] - ref_iso["p_tok"][drows]).max())
            rep["q_err"] = float(np.abs(q_g[drows] - ref_iso["q_tok"][drows]).max())
            assert rep["p_err"] < PROB_TOL and rep["q_err"] < PROB_TOL, rep
            # a position the GPU reached must have used the same uniform
            assert np.array_equal(u_g[drows], ref_iso["u"][drows])
    rep["iso_ties"], rep["iso_cdf_ties"] = compare_decisions(case, acc, nxt, ref_iso, CDF_TIE_TOL, "isolated")

    # (ii) end to end: the oracle's own attention -> bf16 -> LM head -> decisions
    ref_e2e = case.oracle_accept(logits_o, top_p=top_p, top_k=top_k, temperatures=temperatures)
    e2e = compare_end_to_end(case, acc, nxt, ref_e2e, ref_iso, logits_o, logits_g, t, top_p, top_k=top_k,
                             temperatures=temperatures)
    rep["e2e_ties"], rep["e2e_cdf_ties"] = e2e["ties"], e2e["cdf_ties"]
    rep["e2e_explained"] = e2e["explained_accept"] + e2e["explained_token"]
    if case.mode == 0 and drows.size:
        rep["p_err_e2e"] = float(np.abs(dbg["p_tok"].cpu().numpy()[drows] - ref_e2e["p_tok"][drows]).max())
    rep["accepted_len"] = acc
    rep["next_token"] = nxt
    rep["oracle_accepted_len"] = ref_e2e["accepted_len"]
    return rep
