"""Host-side channel-aware drafting policy of the paper (Section IV-B, Algorithm 2 Steps 1 and 3).

This is what makes draft lengths ragged on the cloud side: every edge device picks its stride K_n
from its current uplink rate, so a verification batch mixes many K.  Nothing here runs on the GPU;
it turns a measured verification cost (T_base, delta_cloud from ``bench.py --fit-k``) into strides,
traces of draft lengths and the effective token generation rate the paper optimises.

Notation follows the paper: K stride, R_n uplink rate (bit/s), b bits per token index, O_header
protocol overhead (bits), T_prop one-way propagation delay, alpha_edge / beta edge drafting cost,
T_base / delta_cloud cloud verification cost, T_down downlink latency, gamma_hat acceptance estimate.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Iterable, List, Sequence

import numpy as np


@dataclass
class LatencyModel:
    """Refined latency model: T_step(K, R) = T_edge(K) + T_up(K, R) + T_cloud(K) + T_down."""
    alpha_edge: float            # s per drafted token
    beta_edge: float             # s, fixed edge cost per step
    t_prop: float                # s, one-way propagation (half the round-trip time)
    bits_per_token: float        # b
    header_bits: float           # O_header
    t_base: float                # s, cloud verification, fixed part
    delta_cloud: float           # s per verified draft token
    t_down: float                # s

    def t_edge(self, k):
        return self.alpha_edge * k + self.beta_edge

    def t_up(self, k, rate):
        return self.t_prop + (k * self.bits_per_token + self.header_bits) / rate

    def t_cloud(self, k):
        return self.t_base + k * self.delta_cloud

    def t_step(self, k, rate):
        return self.t_edge(k) + self.t_up(k, rate) + self.t_cloud(k) + self.t_down

    def t_marginal(self, rate):
        """Cost of one more drafted token (Algorithm 2): alpha_edge + b / R_n + delta_cloud."""
        return self.alpha_edge + self.bits_per_token / rate + self.delta_cloud

    def t_fixed(self, rate):
        """Everything in T_step that does not grow with K."""
        return self.beta_edge + self.t_prop + self.header_bits / rate + self.t_base + self.t_down


def expected_accepted(k, gamma: float, model: str = "geometric"):
    """E[tau | K].  'linear' is the gamma_hat * K of Algorithm 2; 'geometric' is the decay model of
    Section IV-B (draft j is reached only if all earlier ones were accepted): sum_{j=1..K} gamma^j."""
    k = np.asarray(k, dtype=np.float64)
    if model == "linear":
        return gamma * k
    if model == "geometric":
        if gamma >= 1.0:
            return k
        return gamma * (1.0 - gamma ** k) / (1.0 - gamma)
    raise ValueError(model)


def optimal_stride(rate: float, gamma: float, lat: LatencyModel, k_max: int, model: str = "geometric") -> int:
    """K_n* = argmax_{1 <= K <= K_max} (1 + E[tau | K]) / (T_fixed + K * T_marginal(n)); ties to the smaller K."""
    ks = np.arange(1, k_max + 1)
    etgr = (1.0 + expected_accepted(ks, gamma, model)) / (lat.t_fixed(rate) + ks * lat.t_marginal(rate))
    return int(ks[int(np.argmax(etgr))])


def ema_update(gamma_hat: float, tau: int, k: int, mu: float) -> float:
    """Algorithm 2, Step 3: gamma_hat <- (1 - mu) * gamma_hat + mu * tau / K."""
    return (1.0 - mu) * gamma_hat + mu * (tau / k)


def simulate(rates: Iterable[float], lat: LatencyModel, true_gamma: float, k_max: int = 12, mu: float = 0.1,
             gamma0: float = 0.8, model: str = "geometric", fixed_k: int | None = None, seed: int = 0):
    """One user's decoding loop over a trace of uplink rates.  Acceptance of each draft token is an
    independent Bernoulli(true_gamma) until the first rejection.  Returns the strides, the accepted
    counts and the effective token generation rate sum(tau + 1) / sum(T_step)."""
    rng = np.random.RandomState(seed)
    gamma_hat = gamma0
    ks: List[int] = []
    taus: List[int] = []
    t_total = 0.0
    for rate in rates:
        k = fixed_k if fixed_k is not None else optimal_stride(rate, gamma_hat, lat, k_max, model)
        acc = rng.random_sample(k) < true_gamma
        tau = int(k if acc.all() else np.argmin(acc))
        gamma_hat = ema_update(gamma_hat, tau, k, mu)
        t_total += lat.t_step(k, rate)
        ks.append(k)
        taus.append(tau)
    tokens = int(np.sum(taus)) + len(ks)
    return {"k": np.array(ks, np.int32), "tau": np.array(taus, np.int32), "etgr": tokens / t_total,
            "gamma_hat": gamma_hat}


def draft_len_trace(rates_per_user: Sequence[Sequence[float]], lat: LatencyModel, gammas: Sequence[float],
                    k_max: int = 12, **kw) -> np.ndarray:
    """Ragged draft lengths of a verification batch over time: [steps][users]."""
    cols = [simulate(r, lat, g, k_max=k_max, seed=i, **kw)["k"] for i, (r, g) in enumerate(zip(rates_per_user, gammas))]
    return np.stack(cols, axis=1)


# ------------------------------------------------------------------ link traces and the ETGR table

#: stylised uplinks (bit/s): median rate, log-normal spread, probability and depth of a fade per step.
#: They stand in for the 5G / 4G / WiFi conditions of the paper's evaluation (Section V), whose traces are not public.
LINKS = {
    "5g": dict(median=50e6, sigma=0.35, fade_prob=0.02, fade_factor=0.05),
    "4g": dict(median=8e6, sigma=0.50, fade_prob=0.05, fade_factor=0.03),
    "wifi": dict(median=1.5e6, sigma=0.80, fade_prob=0.15, fade_factor=0.02),
}


def link_rate_trace(kind: str, steps: int, seed: int = 0) -> np.ndarray:
    """A seeded trace of uplink rates R_n (bit/s): an AR(1) log-normal around the link's median with
    occasional deep fades (the weak-signal regime in which the paper's policy shortens or lengthens K)."""
    cfg = LINKS[kind]
    rng = np.random.RandomState(seed)
    x = np.zeros(steps)
    for n in range(1, steps):
        x[n] = 0.8 * x[n - 1] + rng.standard_normal() * cfg["sigma"] * 0.6
    rate = cfg["median"] * np.exp(x)
    fades = rng.random_sample(steps) < cfg["fade_prob"]
    rate[fades] *= cfg["fade_factor"]
    return rate


def default_latency_model(t_base_s: float = 232e-6, delta_cloud_s: float = 8.4e-6) -> LatencyModel:
    """Edge and link constants of the order the paper reports (Table V: 8.5 .. 12 ms per drafted token on
    a phone- or Jetson-class device; end-to-end latencies of a few hundred ms, so tens of ms each way),
    with the cloud constants measured by this library."""
    return LatencyModel(alpha_edge=8.5e-3, beta_edge=2e-3, t_prop=40e-3, bits_per_token=17.0, header_bits=400.0,
                        t_base=t_base_s, delta_cloud=delta_cloud_s, t_down=40e-3)


def etgr_table(lat: LatencyModel, gamma: float = 0.7, steps: int = 400, k_max: int = 12,
               fixed=(1, 3, 5, 7), seed: int = 0):
    """Effective token generation rate (Eq. 2: tokens committed per second of wall time) of the adaptive
    stride against fixed strides, per link kind -- the comparison of the paper's stride ablation."""
    out = {}
    for i, kind in enumerate(LINKS):
        rates = link_rate_trace(kind, steps, seed + i)
        row = {"adaptive": simulate(rates, lat, gamma, k_max=k_max, seed=seed)["etgr"]}
        row["mean_k_adaptive"] = float(simulate(rates, lat, gamma, k_max=k_max, seed=seed)["k"].mean())
        for k in fixed:
            row[f"fixed_{k}"] = simulate(rates, lat, gamma, k_max=k_max, fixed_k=k, seed=seed)["etgr"]
        out[kind] = row
    return out


def batch_draft_lengths(batch: int, lat: LatencyModel, k_max: int = 12, seed: int = 0, warm_steps: int = 30):
    """Draft lengths of one verification batch as the policy produces them: user b sits on a 5G, 4G or
    WiFi-like link (round-robin), has its own true acceptance rate in 0.4 .. 0.9, and has run the policy
    for warm_steps steps (so its EMA has left the prior); the stride it picks at the next step is its k_b."""
    kinds = list(LINKS)
    rng = np.random.RandomState(seed)
    ks = np.zeros(batch, np.int32)
    gammas = rng.uniform(0.4, 0.9, batch)
    for b in range(batch):
        rates = link_rate_trace(kinds[b % len(kinds)], warm_steps + 1, seed * 1000 + b)
        sim = simulate(rates[:warm_steps], lat, float(gammas[b]), k_max=k_max, seed=seed * 1000 + b)
        ks[b] = optimal_stride(float(rates[warm_steps]), sim["gamma_hat"], lat, k_max)
    return ks, gammas
