"""Seeded synthetic inputs shaped like the BitRL backbone's BitLinear workloads.

This module holds no arithmetic of the method: it only draws random numbers.  Both the CUDA library's
tests/benchmarks and the CPU oracle's tests take their inputs from here, so that the two sides see the
same bytes.  Everything is generated on the CPU with ``torch.Generator`` and returned as CPU tensors.

Recipe (stands in for the real BitNet b1.58 weights and real serialized-state activations, which are not
available offline):
  * master weights: fp32, N(0, sigma=0.02), shape [N_out, K_in];
  * activations: N(0,1) fp32; a fixed 1 % of the K channels (chosen by a seeded permutation) is
    multiplied by 20 to imitate outlier channels; the result is cast to bf16;
  * states: 15-40 tokens each (uniform), the range the paper reports for serialized states.
"""
from __future__ import annotations

import torch

SIGMA_W = 0.02
OUTLIER_FRACTION = 0.01
OUTLIER_SCALE = 20.0

# (K_in, N_out) of the four BitLinear matrices of one ~2B BitNet b1.58 block.
BLOCK_SHAPES = {
    "qkv": (2560, 3840),
    "out": (2560, 2560),
    "gateup": (2560, 13824),
    "down": (6912, 2560),
}
ENCODER = {"d": 2560, "d_ff": 6912, "n_heads": 20, "n_kv_heads": 5, "n_layers": 30}


def _gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    return g


def master_weights(N: int, K: int, seed: int) -> torch.Tensor:
    """fp32 [N,K] ~ N(0, 0.02)."""
    return torch.randn(N, K, generator=_gen(seed), dtype=torch.float32) * SIGMA_W


def activations(M: int, K: int, seed: int, outliers: bool = True, outlier_seed: int = 3000) -> torch.Tensor:
    """bf16 [M,K] ~ N(0,1), optionally with floor(0.01*K) channels scaled by 20."""
    x = torch.randn(M, K, generator=_gen(seed), dtype=torch.float32)
    if outliers:
        n_out = int(OUTLIER_FRACTION * K)
        if n_out > 0:
            perm = torch.randperm(K, generator=_gen(outlier_seed))
            x[:, perm[:n_out]] *= OUTLIER_SCALE
    return x.to(torch.bfloat16)


def encoder_layer_weights(layer: int, seed: int = 5000, dims: dict | None = None):
    """The four master matrices (qkv, out, gateup, down) of one block; matrix j of layer l uses seed+4l+j."""
    e = dict(ENCODER if dims is None else dims)
    d, d_ff = e["d"], e["d_ff"]
    hd = d // e["n_heads"]
    n_qkv = d + 2 * e["n_kv_heads"] * hd
    shapes = [(n_qkv, d), (d, d), (2 * d_ff, d), (d, d_ff)]
    return [master_weights(n, k, seed + 4 * layer + j) for j, (n, k) in enumerate(shapes)]


STATE_TOKENS_MIN, STATE_TOKENS_MAX = 15, 40  # tokens per serialized state (the range the paper reports, Sec. V)


def state_offsets(n_states: int, seed: int, lo: int = STATE_TOKENS_MIN, hi: int = STATE_TOKENS_MAX) -> torch.Tensor:
    """Token offsets [n_states+1] (int64, CPU) of states whose lengths are uniform integers in [lo, hi]."""
    lens = torch.randint(lo, hi + 1, (n_states,), generator=_gen(seed), dtype=torch.int64)
    return torch.cat([torch.zeros(1, dtype=torch.int64), torch.cumsum(lens, 0)])


HEAD_HIDDEN = (256, 128)  # hidden widths of the policy and value heads (paper: Table VI)


def head_weights(d: int, n_out: int, seed: int, hidden=HEAD_HIDDEN):
    """fp32 (W1t [d,H1], b1, W2t [H1,H2], b2, W3t [H2,n_out], b3), N(0, 1/fan_in) weights and N(0, 0.1) biases."""
    g = _gen(seed)
    dims = [d, hidden[0], hidden[1], n_out]
    out = []
    for i in range(3):
        out.append(torch.randn(dims[i], dims[i + 1], generator=g, dtype=torch.float32) / dims[i] ** 0.5)
        out.append(torch.randn(dims[i + 1], generator=g, dtype=torch.float32) * 0.1)
    return tuple(out)


def rollout(T: int, E: int, seed: int, done_prob: float = 0.02):
    """fp32 rewards [T,E] ~ N(0,1), values [T+1,E] ~ N(0,1), dones [T,E] in {0,1} with P(done) = done_prob."""
    g = _gen(seed)
    r = torch.randn(T, E, generator=g, dtype=torch.float32)
    v = torch.randn(T + 1, E, generator=g, dtype=torch.float32)
    d = (torch.rand(T, E, generator=g) < done_prob).to(torch.float32)
    return r, v, d


def ppo_batch(B: int, A: int, seed: int):
    """logits fp32 [B,A] ~ 2 N(0,1); actions int32 [B]; old_logp = log-softmax of perturbed logits at the action;
    advantages, values, returns fp32 [B] ~ N(0,1)."""
    g = _gen(seed)
    logits = torch.randn(B, A, generator=g, dtype=torch.float32) * 2.0
    actions = torch.randint(0, A, (B,), generator=g, dtype=torch.int32)
    old = torch.log_softmax(logits + 0.3 * torch.randn(B, A, generator=g, dtype=torch.float32), dim=1)
    old_logp = old[torch.arange(B), actions.long()].contiguous()
    adv, v, R = (torch.randn(B, generator=g, dtype=torch.float32) for _ in range(3))
    return logits, actions, old_logp, adv, v, R


def bf16_bits(t: torch.Tensor):
    """bf16 CPU tensor -> numpy uint16 bit patterns (same shape)."""
    assert t.dtype == torch.bfloat16
    return t.contiguous().view(torch.int16).numpy().view("uint16")


def bits_to_bf16(a) -> torch.Tensor:
    """numpy uint16 bit patterns -> bf16 CPU tensor."""
    import numpy as np

    return torch.from_numpy(np.ascontiguousarray(a).view("int16")).view(torch.bfloat16)
