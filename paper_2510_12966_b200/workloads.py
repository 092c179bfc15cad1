"""Seeded synthetic inputs for the verification path. Holds no arithmetic of the method itself.

The paper evaluates on CSQA prompts with Llama-3.2-1B / 3.2-3B / 3.1-8B (Sec. 4.1); neither the prompts
nor the weights are used here. These generators stand in for that workload: logits tensors with the
Llama-3-family vocabulary sizes and the paper's speculative-length / threshold ranges, built from a
common recipe:

    z_target ~ N(0, 3^2) i.i.d. per entry, plus ``boost`` on one uniformly chosen token per position;
    z_qual   = z_target + N(0, sigma_q^2);   z_draft = z_target + N(0, sigma_d^2);
    draft tokens ~ softmax(z_draft) (drawn by torch.multinomial, the harness's own sampler).

Everything is rounded to the run dtype before use, and both the CUDA library and the CPU oracle are
fed the same bit patterns. Generator seed = 1000 * config + round.
"""
from __future__ import annotations

import dataclasses
from typing import Optional, Tuple

import numpy as np
import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    kind: str                      # "stage" | "pyramid" | "fused"
    B: int
    V: int
    dtype: str                     # "f32" | "bf16"
    K_d: int
    K_q: int                       # == K_d for single-stage workloads
    rounds: int
    boost: Tuple[float, float]     # (lo, hi): per-sequence boost ~ U[lo, hi]; lo == hi means constant
    sigma_q: float
    sigma_d: float
    tau_q: float
    tau_t: float
    d_model: int = 0               # fused workload only


CONFIGS = {
    1: Workload("cfg1_tiny_fp32", "stage", B=1, V=32000, dtype="f32", K_d=4, K_q=4, rounds=64,
                boost=(8.0, 8.0), sigma_q=0.0, sigma_d=1.0, tau_q=0.3, tau_t=0.3),
    2: Workload("cfg2_single_stream", "pyramid", B=1, V=128256, dtype="bf16", K_d=8, K_q=4, rounds=1024,
                boost=(8.0, 8.0), sigma_q=0.7, sigma_d=1.5, tau_q=0.4, tau_t=0.2),
    3: Workload("cfg3_batched_serving", "pyramid", B=64, V=128256, dtype="bf16", K_d=16, K_q=8, rounds=256,
                boost=(4.0, 12.0), sigma_q=0.7, sigma_d=1.5, tau_q=0.4, tau_t=0.2),
    4: Workload("cfg4_large_vocab_sweep", "pyramid", B=256, V=152064, dtype="bf16", K_d=8, K_q=4, rounds=1,
                boost=(8.0, 8.0), sigma_q=0.5, sigma_d=2.0, tau_q=0.2, tau_t=0.2),
    5: Workload("cfg5_fused_lmhead", "fused", B=32, V=128256, dtype="bf16", K_d=8, K_q=8, rounds=1,
                boost=(0.0, 0.0), sigma_q=0.7, sigma_d=0.0, tau_q=0.2, tau_t=0.2, d_model=4096),
}
CFG4_K = (4, 8, 16, 32)
CFG4_TAU = (0.05, 0.2, 0.5, 1.0)


def torch_dtype(name: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _target_logits(B, K, V, boost, g, device):
    z = torch.randn((B, K, V), generator=g, device=device, dtype=torch.float32) * 3.0
    lo, hi = boost
    amp = torch.rand((B, 1, 1), generator=g, device=device, dtype=torch.float32) * (hi - lo) + lo
    peak = torch.randint(0, V, (B, K, 1), generator=g, device=device)
    z.scatter_add_(2, peak, amp.expand(B, K, 1).contiguous())
    return z


def _sample_tokens(z, g):
    B, K, V = z.shape
    probs = torch.softmax(z.float().reshape(B * K, V), dim=-1)
    return torch.multinomial(probs, 1, generator=g).reshape(B, K).to(torch.int32)


def make_stage_inputs(B, K, V, dtype="f32", seed=0, boost=(8.0, 8.0), sigma=1.0, device="cpu"):
    """Single-stage inputs: (logits_small, logits_large, draft_tokens); small = large + N(0, sigma^2)."""
    g = _gen(seed, device)
    dt = torch_dtype(dtype)
    z_l = _target_logits(B, K, V, boost, g, device)
    z_s = z_l + torch.randn((B, K, V), generator=g, device=device, dtype=torch.float32) * sigma
    z_l, z_s = z_l.to(dt), z_s.to(dt)
    tok = _sample_tokens(z_s, g)
    return z_s.contiguous(), z_l.contiguous(), tok.contiguous()


def make_pyramid_inputs(B, K_d, K_q, V, dtype="bf16", seed=0, boost=(8.0, 8.0), sigma_q=0.7, sigma_d=1.5,
                        device="cpu"):
    """Two-stage inputs: (logits_draft [B,K_d,V], logits_qual [B,K_d,V], logits_target [B,K_q,V], tokens)."""
    g = _gen(seed, device)
    dt = torch_dtype(dtype)
    z_t = _target_logits(B, K_d, V, boost, g, device)
    z_q = (z_t + torch.randn((B, K_d, V), generator=g, device=device, dtype=torch.float32) * sigma_q).to(dt)
    z_d = (z_t + torch.randn((B, K_d, V), generator=g, device=device, dtype=torch.float32) * sigma_d).to(dt)
    z_t = z_t[:, :K_q].to(dt).contiguous()
    tok = _sample_tokens(z_d, g)
    return z_d.contiguous(), z_q.contiguous(), z_t, tok.contiguous()


def make_fused_inputs(B, K, V, d_model, seed=0, sigma_q=0.7, device="cpu"):
    """Fused-LM-head inputs: hidden [B*K, d] bf16 ~ N(0,1); the LM-head weight ~ N(0, 0.02^2) bf16 in the
    layout checkpoints keep it in, w_t [V, d] (out x in; the [d, V] matrix of the config is its transpose);
    qualifier logits [B, K, V] bf16 = hidden x W + N(0, sigma_q^2) (a library matmul builds this input,
    nothing more); window tokens drawn from the qualifier's softmax."""
    g = _gen(seed, device)
    h = torch.randn((B * K, d_model), generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)
    w_t = (torch.randn((V, d_model), generator=g, device=device, dtype=torch.float32) * 0.02).to(torch.bfloat16)
    z = h.float() @ w_t.float().T
    z_q = (z + torch.randn((B * K, V), generator=g, device=device, dtype=torch.float32) * sigma_q)
    z_q = z_q.to(torch.bfloat16).reshape(B, K, V).contiguous()
    tok = _sample_tokens(z_q, g)
    return h.contiguous(), w_t.contiguous(), z_q, tok.contiguous()


def workload_inputs(cfg: int, round_idx: int = 0, device="cpu", B: Optional[int] = None,
                    K_d: Optional[int] = None, K_q: Optional[int] = None, V: Optional[int] = None):
    """Inputs of workload configuration ``cfg`` for one round; B / K / V can be overridden for reduced test cases."""
    w = CONFIGS[cfg]
    B = w.B if B is None else B
    K_d = w.K_d if K_d is None else K_d
    K_q = w.K_q if K_q is None else K_q
    V = w.V if V is None else V
    seed = 1000 * cfg + round_idx
    if w.kind == "stage":
        return make_stage_inputs(B, K_d, V, w.dtype, seed, w.boost, w.sigma_d, device)
    if w.kind == "pyramid":
        return make_pyramid_inputs(B, K_d, K_q, V, w.dtype, seed, w.boost, w.sigma_q, w.sigma_d, device)
    return make_fused_inputs(B, K_d, V, w.d_model, seed, w.sigma_q, device)


def to_host_bits(t: torch.Tensor) -> np.ndarray:
    """Host numpy view for the oracle: float32 as is, bf16 as its uint16 bit patterns, ints unchanged."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def shard_batch(B: int, rank: int, world_size: int) -> Tuple[int, int]:
    """Contiguous batch slice [lo, hi) of sequences owned by ``rank``; sequences are independent."""
    base, rem = divmod(B, world_size)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


def shard_call(B: int, rank: int, world_size: int) -> Tuple[int, int, int]:
    """What ``rank`` hands to a verification call on its shard of a batch of B sequences: the slice [lo, hi) of
    every per-sequence tensor and the ``seq_index_base`` (= lo) that keeps each sequence's random draws those of
    the unsharded call."""
    lo, hi = shard_batch(B, rank, world_size)
    return lo, hi, lo
