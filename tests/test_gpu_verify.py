"""GPU parity of the whole verification step (flexspec_verify through the C ABI) against the
oracle on reduced cases, every sequence compared: peaked logits, ragged batches, greedy mode,
top-p, degenerate drafts, bad inputs, the host-memory entry point.  (The five paper-shaped
workloads at full size are in test_gpu_0_configs.py, which runs first.)"""
import numpy as np
import pytest
import torch

from paper_2601_00644_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _H():
    import tests.harness as H
    return H


def _run(shape, check=None, mode=0, top_p=1.0):
    H = _H()
    case = H.Case(shape, check_seqs=check, mode=mode)
    case.build_drafts()
    ver = H.make_verifier(case)
    if top_p < 1.0:
        ver.set_top_p(top_p)
    rep = H.full_parity(case, ver, top_p=top_p)
    # same call again: identical outputs (tickets reset, no stale state)
    acc2, nxt2 = H.run_gpu_verify(case, ver)
    assert np.array_equal(acc2, rep["accepted_len"]) and np.array_equal(nxt2, rep["next_token"])
    ver.close()
    return case, rep


def _few_differences(case, rep, share=0.05):
    """Every end-to-end difference has been shown by the harness to be a near-tie or covered by the
    distance between the two logit sets; on top of that they must stay rare: at most `share` of the
    decisions taken (acceptance tests + emitted tokens), plus one."""
    decisions = int(sum(case.k[b] + 1 for b in case.check))
    n = rep["e2e_ties"] + rep["e2e_cdf_ties"] + rep["e2e_explained"]
    assert n <= 1 + int(share * decisions), rep


def test_tiny_shape_greedy_and_peaked():
    shape = wl.CONFIGS["tiny"]
    _run(shape, mode=1)
    case, rep = _run(wl.peaked(shape))
    _few_differences(case, rep)


def test_reduced_8b_shape_flat_and_peaked():
    base = wl.scaled(wl.CONFIGS["llama3_8b"], batch=3, vocab=20000, ctx_min=700, ctx_max=700, index=11)
    case, rep = _run(base)
    assert rep["e2e_ties"] + rep["e2e_cdf_ties"] + rep["e2e_explained"] <= 1
    # peaked logits: a bf16 rounding of the attention output that falls the other way moves a logit by
    # ~1e-2, so an end-to-end decision may differ -- but only where the oracle itself shows that the
    # logit difference covers its margin (harness.compare_end_to_end); the isolated comparison is exact
    case, rep = _run(wl.peaked(base))
    assert rep["iso_ties"] + rep["iso_cdf_ties"] <= 1
    _few_differences(case, rep)


def test_verify_with_top_p_on_peaked_logits():
    """The whole step with nucleus sampling (the paper's stochastic regime, top-p 0.9): decisions against
    the oracle fed the GPU's own logits, and end to end under the same rule as the unfiltered tests (a
    token that enters or leaves the nucleus between the two logit sets shows up in the emission weights)."""
    shape = wl.peaked(wl.scaled(wl.CONFIGS["llama3_8b"], batch=4, vocab=20000, ctx_min=300, ctx_max=700, index=16))
    case, rep = _run(shape, top_p=0.9)
    assert rep["topp_ties"] <= 1
    # a token that enters or leaves a nucleus renormalises the whole row, so more decisions move
    _few_differences(case, rep, share=0.2)


def test_verify_with_top_k_and_per_sequence_temperatures():
    """The whole step with top-k 20 (then top-p 0.95) and a temperature of its own for every sequence: the
    LM-head epilogue, the draft-logit statistics, the filter and the acceptance kernel all use the
    sequence's temperature."""
    H = _H()
    shape = wl.peaked(wl.scaled(wl.CONFIGS["llama3_8b"], batch=5, vocab=20000, ctx_min=200, ctx_max=500, k_min=2, k_max=6,
                                index=18))
    case = H.Case(shape)
    temps = np.array([0.6, 1.0, 1.4, 0.8, 1.1])
    # the edge draws its tokens at the sequence's temperature too: rebuild the drafts row by row
    case.build_drafts()
    for b in range(case.batch):
        sl = slice(case.tok0[b], case.tok0[b + 1])
        case.draft_tokens[sl] = wl.draw_draft_tokens(case.draft_logits[sl], float(temps[b]), case.inp.token_uniforms[sl])
    ver = H.make_verifier(case)
    t_dev = torch.from_numpy(temps.astype(np.float32)).cuda()
    ver.set_sampling(top_p=0.95, top_k=20, temperatures=t_dev)
    rep = H.full_parity(case, ver, top_p=0.95, top_k=20, temperatures=temps)
    assert rep["topp_ties"] <= 1
    _few_differences(case, rep, share=0.2)
    ver.close()


def test_ragged_batch_with_k0_and_greedy():
    shape = wl.scaled(wl.CONFIGS["adaptive_k"], batch=7, vocab=9000, k_min=0, k_max=12, ctx_min=30,
                      ctx_max=900, index=12)
    _run(shape)
    _run(shape, mode=1)


def test_many_short_sequences_in_one_call():
    """More sequences than threads in a CTA (the per-CTA range computation then handles several
    sequences per thread), tiny contexts, k from 0: every sequence against the oracle."""
    shape = wl.scaled(wl.CONFIGS["tiny"], batch=300, vocab=1000, k_min=0, k_max=3, ctx_min=0, ctx_max=40, index=17)
    case, rep = _run(wl.peaked(shape))
    assert rep["iso_ties"] + rep["iso_cdf_ties"] <= 2
    # ~750 decisions on peaked logits (the bf16 probabilities of the second attention product move a
    # logit by up to 4e-3 of the row's scale): a few percent of them sit where that decides
    _few_differences(case, rep)
    case, rep = _run(wl.peaked(shape), mode=1)
    _few_differences(case, rep)


def test_degenerate_cases_p_equals_q_and_disjoint_support():
    """Long-context config's sub-cases on a reduced shape: a sequence whose draft logits are the
    target's own (every draft accepted) and one whose drafts lie outside the target's support
    (rejected at position 0, emitted token from p)."""
    H = _H()
    shape = wl.scaled(wl.CONFIGS["long_ctx"], batch=3, vocab=12000, ctx_min=3000, ctx_max=3000,
                      k_min=6, k_max=6, index=13)
    case = H.Case(shape)
    case.build_drafts()
    ver = H.make_verifier(case)
    inp = case.inp
    # phase 1: the GPU's own target logits
    ver.attention(inp.kv_pages, inp.page_table, inp.kv_len, inp.kv_len.cpu(), inp.hidden,
                  inp.draft_len, inp.draft_len.cpu(), attn_out=None)
    attn = ver.attention(inp.kv_pages, inp.page_table, inp.kv_len, inp.kv_len.cpu(), inp.hidden,
                         inp.draft_len, inp.draft_len.cpu())
    logits = ver.lm_head(attn)
    kk = 6
    # sequence 0: q == p bit for bit
    case.draft_logits[case.tok0[0]:case.tok0[0] + kk] = logits[case.row0[0]:case.row0[0] + kk]
    # sequence 1: drafts on odd ids, the target restricted to even ids
    case.draft_tokens[case.tok0[1]:case.tok0[1] + kk] = torch.tensor([1, 3, 5, 7, 9, 11], dtype=torch.int32, device="cuda")
    words = (shape.vocab + 31) // 32
    mask = np.full((3, words), 0xFFFFFFFF, np.uint32)
    mask[1] = 0x55555555
    mask_dev = torch.from_numpy(mask.view(np.int32)).cuda()
    acc, nxt = H.run_gpu_verify(case, ver, vocab_mask_dev=mask_dev)
    assert acc[0] == kk
    assert acc[1] == 0 and nxt[1] % 2 == 0
    # oracle on the same inputs (its own logits; masks applied identically)
    case.vocab_mask = mask
    _, _, logits_o = case.oracle_front()
    ref = case.oracle_accept(logits_o)
    assert ref["accepted_len"][1] == 0 and ref["next_token"][1] % 2 == 0
    ref_iso = case.oracle_accept(logits.cpu().numpy().astype(np.float64))
    assert ref_iso["accepted_len"][0] == kk
    H.compare_decisions(case, acc, nxt, ref_iso, H.CDF_TIE_TOL, "degenerate")
    ver.close()


def test_bad_inputs_are_reported_not_faulted():
    H = _H()
    from paper_2601_00644_b200 import binding as B
    shape = wl.scaled(wl.CONFIGS["tiny"], index=14)
    case = H.Case(shape)
    case.build_drafts()
    ver = H.make_verifier(case)
    inp = case.inp
    args = dict(kv_pages=inp.kv_pages, page_table=inp.page_table, kv_len=inp.kv_len, kv_len_host=inp.kv_len.cpu(),
                hidden=inp.hidden, draft_tokens=case.draft_tokens, draft_logits=case.draft_logits,
                draft_len=inp.draft_len, draft_len_host=inp.draft_len.cpu(), seeds=inp.seeds)
    # host-side rejections
    with pytest.raises(B.FlexSpecError) as e:
        ver.verify(**{**args, "draft_len_host": torch.tensor([9], dtype=torch.int32)})
    assert e.value.code == B.ERR_INVALID_ARG
    with pytest.raises(B.FlexSpecError):
        ver.verify(**{**args, "kv_len_host": torch.tensor([2], dtype=torch.int32)})
    with pytest.raises(B.FlexSpecError):
        ver.verify(**{**args, "draft_logits": None})
    with pytest.raises(B.FlexSpecError):
        ver.verify(**{**args, "temperature": -1.0})
    # draft logits that do not start on a 16-byte boundary (vocab is a multiple of four, so the kernels
    # would read them with 16-byte loads): rejected on the host, nothing is launched
    s_rows, vocab = case.draft_logits.shape
    shifted = torch.zeros(s_rows * vocab + 1, dtype=torch.float32, device="cuda")[1:].view(s_rows, vocab)
    assert shifted.data_ptr() % 16 == 4 and shifted.is_contiguous()
    with pytest.raises(B.FlexSpecError) as e:
        ver.verify(**{**args, "draft_logits": shifted})
    assert e.value.code == B.ERR_INVALID_ARG
    # device-side: a page id outside the pool is reported through the status word, no fault
    bad_pt = inp.page_table.clone()
    bad_pt[0, 1] = inp.kv_pages.shape[0] + 5
    ver.verify(**{**args, "page_table": bad_pt})
    torch.cuda.synchronize()
    code, st = ver.status()
    assert code == B.ERR_BAD_PAGE and st[1] == inp.kv_pages.shape[0] + 5
    # a token id outside the vocabulary
    bad_tok = case.draft_tokens.clone()
    bad_tok[2] = shape.vocab + 3
    ver.verify(**{**args, "draft_tokens": bad_tok})
    torch.cuda.synchronize()
    code, st = ver.status()
    assert code == B.ERR_BAD_TOKEN
    # the handle is still usable
    acc, nxt = H.run_gpu_verify(case, ver)
    assert 0 <= acc[0] <= 4
    ver.close()


def test_verify_host_entry_matches_device_entry():
    H = _H()
    shape = wl.scaled(wl.CONFIGS["llama3_8b"], batch=4, vocab=6000, ctx_min=300, ctx_max=400, index=15)
    case = H.Case(shape)
    case.build_drafts()
    ver = H.make_verifier(case)
    acc, nxt = H.run_gpu_verify(case, ver)
    inp = case.inp
    pin = lambda t: t.cpu().pin_memory()
    acc_h = torch.empty(case.batch, dtype=torch.int32).pin_memory()
    nxt_h = torch.empty(case.batch, dtype=torch.int32).pin_memory()
    ver.verify_host(inp.kv_pages, inp.page_table, inp.kv_len.cpu(), pin(inp.hidden), pin(case.draft_tokens),
                    pin(case.draft_logits), pin(inp.draft_len), pin(inp.seeds), acc_h, nxt_h,
                    temperature=shape.temperature)
    assert np.array_equal(acc_h.numpy(), acc) and np.array_equal(nxt_h.numpy(), nxt)
    # with a vocabulary mask (host memory as well): the same as the device entry with the mask on the device
    words = (shape.vocab + 31) // 32
    mask = np.full((case.batch, words), 0xFFFFFFFF, np.uint32)
    mask[1] = 0x55555555
    mask_t = torch.from_numpy(mask.view(np.int32))
    acc_m, nxt_m = H.run_gpu_verify(case, ver, vocab_mask_dev=mask_t.cuda())
    ver.verify_host(inp.kv_pages, inp.page_table, inp.kv_len.cpu(), pin(inp.hidden), pin(case.draft_tokens),
                    pin(case.draft_logits), pin(inp.draft_len), pin(inp.seeds), acc_h, nxt_h,
                    temperature=shape.temperature, vocab_mask=mask_t.pin_memory())
    assert np.array_equal(acc_h.numpy(), acc_m) and np.array_equal(nxt_h.numpy(), nxt_m) and nxt_m[1] % 2 == 0
    ver.close()
