"""Host-side drafting policy (Section IV-B, Algorithm 2 Steps 1 and 3): closed forms and the
qualitative behaviour the paper states."""
import numpy as np

from paper_2601_00644_b200 import policy as P

LAT = P.LatencyModel(alpha_edge=10e-3, beta_edge=2e-3, t_prop=15e-3, bits_per_token=17, header_bits=320,
                     t_base=232e-6, delta_cloud=8.4e-6, t_down=15e-3)


def test_latency_model_adds_up_and_is_affine_in_k():
    r = 1e6
    for k in (1, 5, 9):
        assert np.isclose(LAT.t_step(k, r), LAT.t_fixed(r) + k * LAT.t_marginal(r))
    assert np.isclose(LAT.t_cloud(5), 232e-6 + 5 * 8.4e-6)
    assert np.isclose(LAT.t_up(4, 1e5), 15e-3 + (4 * 17 + 320) / 1e5)


def test_expected_accepted_models():
    assert np.isclose(P.expected_accepted(5, 0.7, "linear"), 3.5)
    g = 0.7
    assert np.isclose(P.expected_accepted(5, g, "geometric"), sum(g ** j for j in range(1, 6)))
    assert np.isclose(P.expected_accepted(4, 1.0, "geometric"), 4.0)


def test_linear_model_optimum_sits_at_an_end_geometric_in_the_interior():
    # (1 + g K) / (F + K m) is monotone in K: the arg-max is 1 or K_max
    for rate in (2e3, 1e5, 1e7):
        k = P.optimal_stride(rate, 0.8, LAT, 12, "linear")
        assert k in (1, 12)
    # with the decay model the optimum is interior; when the per-token uplink cost b / R_n is what the
    # channel changes (no header), a weak link shortens the stride and a strong one lengthens it,
    # as in the paper's figure on the optimal K
    no_header = P.LatencyModel(**{**LAT.__dict__, "header_bits": 0.0})
    ks = [P.optimal_stride(r, 0.8, no_header, 12, "geometric") for r in (200.0, 500.0, 2e3, 2e5, 2e7)]
    assert all(a <= b for a, b in zip(ks, ks[1:])) and ks[0] < ks[-1]
    assert 1 <= ks[0] and ks[-1] < 12
    # a large fixed header does the opposite: at low rates it inflates T_fixed and longer strides amortise it
    ks_h = [P.optimal_stride(r, 0.8, LAT, 12, "geometric") for r in (500.0, 2e3, 2e5)]
    assert ks_h[0] >= ks_h[-1]
    # brute force agreement
    for r in (2e3, 2e5):
        best = max(range(1, 13), key=lambda k: ((1 + P.expected_accepted(k, 0.8)) / LAT.t_step(k, r), -k))
        assert best == P.optimal_stride(r, 0.8, LAT, 12)


def test_ema_update_and_simulation_bookkeeping():
    assert np.isclose(P.ema_update(0.8, 3, 5, 0.1), 0.9 * 0.8 + 0.1 * 0.6)
    rates = np.full(400, 1e5)
    out = P.simulate(rates, LAT, true_gamma=0.7, k_max=8, seed=3)
    assert out["k"].shape == out["tau"].shape == (400,)
    assert np.all(out["tau"] <= out["k"]) and np.all(out["k"] >= 1) and np.all(out["k"] <= 8)
    t = sum(LAT.t_step(int(k), 1e5) for k in out["k"])
    assert np.isclose(out["etgr"], (out["tau"].sum() + 400) / t)
    assert abs(out["gamma_hat"] - np.mean(out["tau"][-100:] / out["k"][-100:])) < 0.25
    # adaptive beats a badly chosen fixed stride on the same trace
    slow = P.simulate(np.full(400, 2e3), LAT, 0.7, k_max=12, seed=3)
    fixed = P.simulate(np.full(400, 2e3), LAT, 0.7, k_max=12, seed=3, fixed_k=12)
    assert slow["etgr"] >= fixed["etgr"] * 0.999
    trace = P.draft_len_trace([rates[:50], np.full(50, 2e3)], LAT, [0.7, 0.5], k_max=12)
    assert trace.shape == (50, 2) and trace.min() >= 1 and trace.max() <= 12


def test_link_traces_and_etgr_table():
    """The three stylised links are seeded and ordered (5G fastest), and on each of them the adaptive
    stride beats the shortest and the longest fixed stride and stays within a few percent of the best one
    (its acceptance estimate, the EMA of tau / K of Algorithm 2, sits below the per-token rate the
    geometric model wants, so it drafts a little short)."""
    from paper_2601_00644_b200 import policy as P
    r5, r4, rw = (P.link_rate_trace(k, 500, seed=3) for k in ("5g", "4g", "wifi"))
    assert np.array_equal(r5, P.link_rate_trace("5g", 500, seed=3))
    assert np.median(r5) > np.median(r4) > np.median(rw) > 0
    tab = P.etgr_table(P.default_latency_model(), gamma=0.7, steps=600)
    for kind, row in tab.items():
        best_fixed = max(v for k, v in row.items() if k.startswith("fixed_"))
        assert row["adaptive"] >= 0.93 * best_fixed, (kind, row)
        assert row["adaptive"] > row["fixed_1"] and row["adaptive"] > row["fixed_7"], (kind, row)
        assert 1.0 <= row["mean_k_adaptive"] <= 12.0


def test_policy_driven_batch_is_ragged_and_seeded():
    from paper_2601_00644_b200 import policy as P, workloads as wl
    ks, gammas = P.batch_draft_lengths(64, P.default_latency_model(), k_max=12, seed=5)
    assert ks.min() >= 1 and ks.max() <= 12 and len(set(ks.tolist())) >= 3
    # users with a better acceptance history draft longer strides on average
    assert ks[gammas > 0.75].mean() > ks[gammas < 0.55].mean()
    shape = wl.scaled(wl.CONFIGS["adaptive_k_policy"], vocab=64, ctx_min=1, ctx_max=8, n_q_heads=2, n_kv_heads=1, head_dim=64)
    a = wl.make_inputs(shape, with_noise=False).draft_len.numpy()
    b = wl.make_inputs(shape, with_noise=False).draft_len.numpy()
    assert np.array_equal(a, b) and len(set(a.tolist())) >= 3
