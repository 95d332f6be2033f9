"""Seeded synthetic inputs for the cloud-side verification step.

This module only draws random tensors and lays them out; it contains none of the
verification arithmetic (no attention, no LM head, no softmax of the target, no
acceptance test), so both the CUDA path and the CPU oracle can be fed from it
without sharing any of the method's code.

The shapes mirror the workloads the paper evaluates (Section V: Llama-3-8B/70B
class targets, contexts of hundreds to thousands of tokens, draft lengths
K = 1..7 and beyond, acceptance 0.18..0.8); datasets and weights are replaced by
seeded normal tensors.  The draft logits of a verification step are assembled
by the harness as  target logits + sigma * noise;  this module supplies the
noise and, given finished draft logits, draws the draft tokens x_j ~ q_j the
way the edge device would (Algorithm 2, Step 1).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np
import torch

MASTER_SEED = 0x26010644
PAGE_SIZE = 16


@dataclass
class VerifyShape:
    """Static description of one verification workload."""
    name: str
    index: int                    # position in the config list (seed offset)
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    vocab: int
    k_min: int                    # draft length range (inclusive); fixed when equal
    k_max: int
    ctx_min: int                  # committed-context range (inclusive)
    ctx_max: int
    sigma_min: float              # std of the draft-logit noise, per sequence
    sigma_max: float
    temperature: float = 1.0
    input_std: float = 0.02       # hidden / KV / W are N(0, input_std)
    w_std: Optional[float] = None  # overrides input_std for W when set
    notes: str = ""

    @property
    def d_model(self) -> int:
        return self.n_q_heads * self.head_dim


def _shape(name, index, **kw) -> VerifyShape:
    return VerifyShape(name=name, index=index, **kw)


#: the five workloads: tiny / 8B-shaped / ragged adaptive-k / 70B-shaped / long context
CONFIGS: Dict[str, VerifyShape] = {
    "tiny": _shape("tiny", 0, batch=1, n_q_heads=8, n_kv_heads=2, head_dim=64, vocab=4096,
                   k_min=4, k_max=4, ctx_min=128, ctx_max=128, sigma_min=0.5, sigma_max=0.5),
    "llama3_8b": _shape("llama3_8b", 1, batch=16, n_q_heads=32, n_kv_heads=8, head_dim=128,
                        vocab=128256, k_min=5, k_max=5, ctx_min=2048, ctx_max=2048,
                        sigma_min=0.77, sigma_max=0.77),
    "adaptive_k": _shape("adaptive_k", 2, batch=64, n_q_heads=32, n_kv_heads=8, head_dim=128,
                         vocab=128256, k_min=1, k_max=12, ctx_min=512, ctx_max=4096,
                         sigma_min=0.2, sigma_max=1.5),
    "llama3_70b": _shape("llama3_70b", 3, batch=32, n_q_heads=64, n_kv_heads=8, head_dim=128,
                         vocab=128256, k_min=8, k_max=8, ctx_min=8192, ctx_max=8192,
                         sigma_min=0.77, sigma_max=0.77),
    # the paper's own targets (Section V: Llama-2-70B is the main model; Table VI adds Mixtral 8x7B): smaller
    # vocabulary, so attention weighs more against the LM head than at the Llama-3 shapes
    "llama2_70b": _shape("llama2_70b", 5, batch=16, n_q_heads=64, n_kv_heads=8, head_dim=128, vocab=32000,
                         k_min=5, k_max=5, ctx_min=2048, ctx_max=2048, sigma_min=0.77, sigma_max=0.77),
    "mixtral_8x7b": _shape("mixtral_8x7b", 6, batch=16, n_q_heads=32, n_kv_heads=8, head_dim=128, vocab=32000,
                           k_min=5, k_max=5, ctx_min=2048, ctx_max=2048, sigma_min=0.77, sigma_max=0.77),
    # the ragged batch with its draft lengths chosen by the paper's channel-aware policy (Section IV-B)
    # instead of uniformly: users on 5G / 4G / WiFi-like links, each with its own acceptance history
    "adaptive_k_policy": _shape("adaptive_k_policy", 7, batch=64, n_q_heads=32, n_kv_heads=8, head_dim=128,
                                vocab=128256, k_min=1, k_max=12, ctx_min=512, ctx_max=4096,
                                sigma_min=0.2, sigma_max=1.5, notes="k from policy"),
    "long_ctx": _shape("long_ctx", 4, batch=8, n_q_heads=32, n_kv_heads=8, head_dim=128,
                       vocab=128256, k_min=16, k_max=16, ctx_min=32768, ctx_max=32768,
                       sigma_min=0.77 * 0.7, sigma_max=0.77 * 0.7, temperature=0.7),
}


def scaled(shape: VerifyShape, **kw) -> VerifyShape:
    """A copy of `shape` with some fields replaced (reduced parity cases)."""
    d = dict(shape.__dict__)
    d.update(kw)
    return VerifyShape(**d)


def peaked(shape: VerifyShape) -> VerifyShape:
    """Same shape, but inputs scaled so the target logits have std of a few units
    (exercises max-subtraction and makes probabilities far from uniform)."""
    return scaled(shape, name=shape.name + "_peaked", input_std=1.0,
                  w_std=4.0 / float(np.sqrt(shape.d_model)))


@dataclass
class VerifyInputs:
    shape: VerifyShape
    draft_len: torch.Tensor        # int32 [B]
    kv_len: torch.Tensor           # int32 [B]   = context + draft_len + 1
    sigma: torch.Tensor            # fp32  [B]
    hidden: torch.Tensor           # bf16  [M, d]
    kv_pages: torch.Tensor         # bf16  [num_pages, 2, Hkv, 16, Dh]
    page_table: torch.Tensor       # int32 [B, max_pages_per_seq], unused slots = -1
    lm_head_w: torch.Tensor        # bf16  [V, d]
    noise: torch.Tensor            # fp32  [S, V], already scaled by sigma_b
    seeds: torch.Tensor            # int64 [B] holding the uint64 bit patterns
    token_uniforms: torch.Tensor   # fp64  [S] in [0,1): the edge's own draws for x_j ~ q_j
    extra: dict = field(default_factory=dict)

    @property
    def batch(self) -> int:
        return int(self.draft_len.numel())

    @property
    def m_rows(self) -> int:
        return int(self.draft_len.sum().item()) + self.batch

    @property
    def s_rows(self) -> int:
        return int(self.draft_len.sum().item())

    def row_offsets(self) -> np.ndarray:
        k = self.draft_len.cpu().numpy().astype(np.int64)
        return np.concatenate([[0], np.cumsum(k + 1)])

    def tok_offsets(self) -> np.ndarray:
        k = self.draft_len.cpu().numpy().astype(np.int64)
        return np.concatenate([[0], np.cumsum(k)])


def _randn_bf16(shape, std, gen, device, chunk_elems=1 << 26):
    """N(0, std) rounded to bf16, drawn in chunks to bound temporary memory."""
    n = int(np.prod(shape))
    out = torch.empty(n, dtype=torch.bfloat16, device=device)
    for lo in range(0, n, chunk_elems):
        hi = min(n, lo + chunk_elems)
        out[lo:hi] = (torch.randn(hi - lo, generator=gen, device=device, dtype=torch.float32)
                      * std).to(torch.bfloat16)
    return out.view(*shape)


def make_inputs(shape: VerifyShape, device: str = "cpu", spare_pages: int = 3,
                with_noise: bool = True) -> VerifyInputs:
    """Draw every tensor of one verification step from the shape's seed."""
    seed = MASTER_SEED + shape.index
    host_rng = np.random.RandomState(seed & 0x7FFFFFFF)
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)

    b = shape.batch
    k = host_rng.randint(shape.k_min, shape.k_max + 1, size=b).astype(np.int32)
    if shape.notes == "k from policy":
        from . import policy
        k, _ = policy.batch_draft_lengths(b, policy.default_latency_model(), k_max=shape.k_max, seed=seed & 0xFFFF)
        k = np.clip(k, shape.k_min, shape.k_max).astype(np.int32)
    ctx = host_rng.randint(shape.ctx_min, shape.ctx_max + 1, size=b).astype(np.int32)
    sigma = host_rng.uniform(shape.sigma_min, shape.sigma_max, size=b).astype(np.float32)
    kv_len = (ctx + k + 1).astype(np.int32)
    seeds = host_rng.randint(0, 2 ** 63 - 1, size=b, dtype=np.int64) * 2 + host_rng.randint(0, 2, size=b)

    pages_per_seq = (kv_len + PAGE_SIZE - 1) // PAGE_SIZE
    max_pages = int(pages_per_seq.max())
    num_pages = int(pages_per_seq.sum()) + spare_pages
    perm = host_rng.permutation(num_pages).astype(np.int32)
    page_table = np.full((b, max_pages), -1, dtype=np.int32)
    cur = 0
    for i in range(b):
        n = int(pages_per_seq[i])
        page_table[i, :n] = perm[cur:cur + n]
        cur += n

    m = int(k.sum()) + b
    s = int(k.sum())
    d = shape.d_model
    w_std = shape.w_std if shape.w_std is not None else shape.input_std
    hidden = _randn_bf16((m, d), shape.input_std, gen, device)
    kv_pages = _randn_bf16((num_pages, 2, shape.n_kv_heads, PAGE_SIZE, shape.head_dim),
                           shape.input_std, gen, device)
    lm_head_w = _randn_bf16((shape.vocab, d), w_std, gen, device)

    if with_noise and s > 0:
        noise = torch.randn(s, shape.vocab, generator=gen, device=device, dtype=torch.float32)
        sig_rows = torch.from_numpy(np.repeat(sigma, k)).to(device)
        noise *= sig_rows[:, None]
    else:
        noise = torch.zeros(s, shape.vocab, dtype=torch.float32, device=device)
    token_uniforms = torch.from_numpy(host_rng.random_sample(s)).to(device)

    return VerifyInputs(
        shape=shape,
        draft_len=torch.from_numpy(k).to(device),
        kv_len=torch.from_numpy(kv_len).to(device),
        sigma=torch.from_numpy(sigma).to(device),
        hidden=hidden, kv_pages=kv_pages,
        page_table=torch.from_numpy(page_table).to(device),
        lm_head_w=lm_head_w, noise=noise,
        seeds=torch.from_numpy(seeds.astype(np.int64)).to(device),
        token_uniforms=token_uniforms,
    )


def draw_draft_tokens(draft_logits: torch.Tensor, temperature: float,
                      token_uniforms: torch.Tensor) -> torch.Tensor:
    """The edge's own sampling x_j ~ softmax(draft_logits_j / T) (Algorithm 2, Step 1),
    by inverse CDF with the supplied uniforms.  int32 [S]."""
    if draft_logits.shape[0] == 0:
        return torch.zeros(0, dtype=torch.int32, device=draft_logits.device)
    q = torch.softmax(draft_logits.double() / temperature, dim=-1)
    cdf = torch.cumsum(q, dim=-1)
    idx = torch.searchsorted(cdf, token_uniforms.double()[:, None], right=True).squeeze(-1)
    return idx.clamp_(max=draft_logits.shape[1] - 1).to(torch.int32)


def bits_u16(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> numpy uint16 bit patterns (host)."""
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def seeds_u64(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().numpy().view(np.uint64)
