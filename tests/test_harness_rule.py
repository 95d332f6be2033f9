"""The end-to-end comparison rule of the GPU parity harness, exercised on the CPU.

`harness.compare_end_to_end` accepts a decision that differs from the oracle's own chain only when
the oracle shows that the difference between the two logit sets covers its margin.  Here the "other
side" is the oracle itself, run on deliberately perturbed logits: genuine flips must be accepted and
counted, a planted wrong decision must fail."""
import numpy as np
import pytest

import oracle
import tests.harness as H
from paper_2601_00644_b200 import workloads as wl


def _case(mode, batch=120, vocab=257, seed_index=31):
    shape = wl.peaked(wl.scaled(wl.CONFIGS["tiny"], batch=batch, vocab=vocab, k_min=0, k_max=4, ctx_min=0,
                                ctx_max=20, index=seed_index))
    case = H.Case(shape, device="cpu", mode=mode)
    case.build_drafts()
    return case


@pytest.mark.parametrize("mode", [0, 1])
def test_flips_caused_by_a_logit_perturbation_are_explained_and_counted(mode):
    case = _case(mode)
    _, _, logits_o = case.oracle_front()
    rng = np.random.RandomState(5)
    # a relative perturbation of the size the tolerance on the logits allows (2e-2 of the row's scale)
    logits_g = (logits_o + rng.standard_normal(logits_o.shape) * 1e-2 * np.abs(logits_o).max()).astype(np.float32)
    ref_own = case.oracle_accept(logits_o)
    ref_g = case.oracle_accept(logits_g.astype(np.float64))
    differ = int(np.sum((ref_own["accepted_len"] != ref_g["accepted_len"]) |
                        (ref_own["next_token"] != ref_g["next_token"])))
    assert differ > 0, "the perturbation is meant to flip a few of the decisions"
    out = H.compare_end_to_end(case, ref_g["accepted_len"], ref_g["next_token"], ref_own, ref_g, logits_o,
                               logits_g, case.shape.temperature)
    assert sum(out.values()) == differ


@pytest.mark.parametrize("mode", [0, 1])
def test_a_wrong_decision_is_not_explained(mode):
    case = _case(mode, batch=30, seed_index=32)
    _, _, logits_o = case.oracle_front()
    logits_g = logits_o.astype(np.float32)                 # same logits up to fp32 rounding
    ref_own = case.oracle_accept(logits_o)
    ref_g = case.oracle_accept(logits_g.astype(np.float64))
    acc = ref_g["accepted_len"].copy()
    nxt = ref_g["next_token"].copy()
    # plant a wrong emitted token in the sequence whose CDF margin is the largest
    b = int(np.argmax(np.where(np.isfinite(ref_own["cdf_margin"]), ref_own["cdf_margin"], -1.0))) if mode == 0 else 3
    nxt[b] = (nxt[b] + 1) % case.shape.vocab
    with pytest.raises(AssertionError):
        H.compare_end_to_end(case, acc, nxt, ref_own, ref_g, logits_o, logits_g, case.shape.temperature)
    # ... and a wrong accepted length
    nxt = ref_g["next_token"].copy()
    kpos = [s for s in range(case.batch) if case.k[s] > 0]
    b = kpos[0]
    acc[b] = (acc[b] + 1) % (case.k[b] + 1)
    with pytest.raises(AssertionError):
        H.compare_end_to_end(case, acc, nxt, ref_own, ref_g, logits_o, logits_g, case.shape.temperature)


def test_emission_weights_match_their_definition():
    rng = np.random.RandomState(9)
    zt = rng.standard_normal(300) * 3
    zd = (zt + rng.standard_normal(300)).astype(np.float32)
    import scipy.special as sp
    p, q = sp.softmax(zt / 0.7), sp.softmax(zd.astype(np.float64) / 0.7)
    r, z = oracle.emission(zt, zd, temperature=0.7)
    assert np.allclose(r, np.maximum(p - q, 0.0), atol=1e-15) and abs(z - np.maximum(p - q, 0.0).sum()) < 1e-14
    r, z = oracle.emission(zt, None, temperature=0.7)
    assert np.allclose(r, p, atol=1e-15) and abs(z - 1.0) < 1e-14
    # the residual of a distribution against itself has no mass: the weights fall back to p
    z32 = zt.astype(np.float32)
    r, z = oracle.emission(z32.astype(np.float64), z32, temperature=1.0)
    assert abs(z - 1.0) < 1e-14 and np.allclose(r, sp.softmax(z32.astype(np.float64)), atol=1e-15)
