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
CDF_TIE_TOL = 1e-6    # inverse-CDF boundary, same logits on both sides: fp32 exponentials (2^-22 rel.) vs fp64


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
    def oracle_accept(self, target_logits_f64, draft_logits=None, draft_tokens=None, temperature=None):
        dl = self.draft_logits if draft_logits is None else draft_logits
        dt = self.draft_tokens if draft_tokens is None else draft_tokens
        t = self.shape.temperature if temperature is None else temperature
        return oracle.accept(self.mode, target_logits_f64,
                             None if dl is None else dl.cpu().numpy(), dt.cpu().numpy(), self.k,
                             self.h_seeds, t, self.vocab_mask, self.check)


def make_verifier(case: Case, debug=True, mode=None):
    from paper_2601_00644_b200 import binding
    s = case.shape
    return binding.Verifier(case.inp.lm_head_w, s.n_q_heads, s.n_kv_heads, s.head_dim,
                            max_batch=case.batch, k_max=max(int(case.k.max()), 1),
                            max_kv_len=int(case.kv_len.max()), mode=case.mode if mode is None else mode,
                            debug=debug)


def run_gpu_verify(case: Case, ver, vocab_mask_dev=None, temperature=None):
    inp = case.inp
    t = case.shape.temperature if temperature is None else temperature
    acc, nxt = ver.verify(inp.kv_pages, inp.page_table, inp.kv_len, inp.kv_len.cpu(), inp.hidden,
                          case.draft_tokens, case.draft_logits, inp.draft_len, inp.draft_len.cpu(),
                          inp.seeds, temperature=t, vocab_mask=vocab_mask_dev)
    torch.cuda.synchronize()
    code, st = ver.status()
    assert code == 0, f"device status {code} {st}"
    return acc.cpu().numpy(), nxt.cpu().numpy()


def compare_decisions(case: Case, acc_gpu, nxt_gpu, ref, cdf_tol, label=""):
    """accepted_len / next_token against an oracle result `ref` on the checked sequences.
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


def full_parity(case: Case, ver, e2e_cdf_tol=1e-6, vocab_mask_dev=None):
    """Stage-by-stage and end-to-end comparison of one verify call.  Returns a report dict."""
    acc, nxt = run_gpu_verify(case, ver, vocab_mask_dev)
    m, s = case.inp.m_rows, case.inp.s_rows
    dbg = ver.debug(m, s)
    a64, a16, logits_o = case.oracle_front()
    rows = case.rows_of(case.check)
    drows = case.drows_of(case.check)
    rep = {}

    attn_g = dbg["attn_out"].float().cpu().numpy()
    rep["attn_row_err"], ok = rel_close(attn_g[rows], a64[rows])
    assert ok and rep["attn_row_err"] < REL_TOL, f"attention: {rep}"

    logits_g = dbg["logits"].cpu().numpy()
    rep["logit_row_err"], ok = rel_close(logits_g[rows], logits_o[rows])
    assert ok and rep["logit_row_err"] < REL_TOL, f"logits: {rep}"

    # (i) decision stage in isolation: the oracle is fed the GPU's own fp32 logits
    if case.mode == 0:
        ref_iso = case.oracle_accept(logits_g.astype(np.float64))
        p_g = dbg["p_tok"].cpu().numpy()
        q_g = dbg["q_tok"].cpu().numpy()
        u_g = dbg["u"].cpu().numpy().astype(np.float64)
        if drows.size:
            rep["p_err"] = float(np.abs(p_g[drows] - ref_iso["p_tok"][drows]).max())
            rep["q_err"] = float(np.abs(q_g[drows] - ref_iso["q_tok"][drows]).max())
            assert rep["p_err"] < PROB_TOL and rep["q_err"] < PROB_TOL, rep
            # a position the GPU reached must have used the same uniform
            assert np.array_equal(u_g[drows], ref_iso["u"][drows])
    else:
        ref_iso = case.oracle_accept(logits_g.astype(np.float64))
    rep["iso_ties"], rep["iso_cdf_ties"] = compare_decisions(case, acc, nxt, ref_iso, CDF_TIE_TOL, "isolated")

    # (ii) end to end: the oracle's own attention -> bf16 -> LM head -> decisions
    ref_e2e = case.oracle_accept(logits_o)
    rep["e2e_ties"], rep["e2e_cdf_ties"] = compare_decisions(case, acc, nxt, ref_e2e, e2e_cdf_tol, "end-to-end")
    if case.mode == 0 and drows.size:
        rep["p_err_e2e"] = float(np.abs(dbg["p_tok"].cpu().numpy()[drows] - ref_e2e["p_tok"][drows]).max())
    rep["accepted_len"] = acc
    rep["next_token"] = nxt
    rep["oracle_accepted_len"] = ref_e2e["accepted_len"]
    return rep
