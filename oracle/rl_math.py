"""CPU oracle of the steps that follow the encoder: the trainable heads, generalized advantage estimation and the
clipped PPO objective.  TEST INFRASTRUCTURE ONLY (same rules as the rest of this package): plain numpy in fp64,
written out term by term, imported only by tests, the smoke check and the benchmark's CPU legs.

Paper anchors
  * Eq. 3: pi(a|s_t) = softmax(g_phi(h_t)), V(s_t) = v_psi(h_t); Table VI: both heads have two hidden layers of
    256 and 128 units and run in fp32.  The paper does not name the activation: tanh is taken (the usual choice
    for PPO heads); the first layer's width follows the latent (d -> 256 -> 128 -> outputs), so the "~50K parameters" the
    paper quotes cannot hold for d = 2560 and the layer widths are followed, not the count.
  * Eq. 1: L_CLIP = E_t[min(r_t A_t, clip(r_t, 1-eps, 1+eps) A_t)], r_t = pi_new(a_t|s_t) / pi_old(a_t|s_t), eps = 0.1.
  * Sec. III-B: entropy regularization with coefficient beta = 0.05; advantages from GAE(lambda = 0.95, gamma = 0.99).
"""
from __future__ import annotations

import numpy as np


def mlp_head(h: np.ndarray, W1t, b1, W2t, b2, W3t, b3) -> np.ndarray:
    """out = (tanh(tanh(h W1t + b1) W2t + b2)) W3t + b3, all fp64.  h [B,d]; W1t [d,H1]; W2t [H1,H2]; W3t [H2,O]."""
    h = np.asarray(h, np.float64)
    a1 = np.tanh(h @ np.asarray(W1t, np.float64) + np.asarray(b1, np.float64))
    a2 = np.tanh(a1 @ np.asarray(W2t, np.float64) + np.asarray(b2, np.float64))
    return a2 @ np.asarray(W3t, np.float64) + np.asarray(b3, np.float64)


def log_softmax(logits: np.ndarray) -> np.ndarray:
    z = np.asarray(logits, np.float64)
    z = z - z.max(axis=-1, keepdims=True)
    return z - np.log(np.exp(z).sum(axis=-1, keepdims=True))


def gae(rewards, values, dones, gamma: float = 0.99, lam: float = 0.95):
    """rewards, dones [T,E]; values [T+1,E] (row T bootstraps).  Backward recursion
         delta_t = r_t + gamma * V_{t+1} * (1 - done_t) - V_t
         A_t     = delta_t + gamma * lam * (1 - done_t) * A_{t+1},  A_T = 0
       Returns (advantages [T,E], returns = advantages + V[:T])."""
    r = np.asarray(rewards, np.float64)
    v = np.asarray(values, np.float64)
    nd = 1.0 - np.asarray(dones, np.float64)
    T, E = r.shape
    adv = np.zeros((T, E), np.float64)
    nxt = np.zeros((E,), np.float64)
    for t in range(T - 1, -1, -1):
        delta = r[t] + gamma * v[t + 1] * nd[t] - v[t]
        nxt = delta + gamma * lam * nd[t] * nxt
        adv[t] = nxt
    return adv, adv + v[:T]


def ppo_loss(logits, actions, old_logp, advantages, values, returns, eps: float = 0.1, beta: float = 0.05):
    """Clipped surrogate (Eq. 1), entropy bonus and value error over a batch of B samples, with the gradients that
    the heads' backward pass starts from.

    Returns a dict: l_clip = mean_t min(r A, clip(r) A); entropy = mean_t H(pi(.|s_t)); policy_loss = -(l_clip + beta *
    entropy); value_loss = mean_t 0.5 (V - R)^2; ratio [B]; dlogits = d policy_loss / d logits [B,A];
    dvalues = d value_loss / d values [B]."""
    z = np.asarray(logits, np.float64)
    B, A = z.shape
    a = np.asarray(actions, np.int64)
    adv = np.asarray(advantages, np.float64)
    logp_all = log_softmax(z)
    p = np.exp(logp_all)
    logp = logp_all[np.arange(B), a]
    ratio = np.exp(logp - np.asarray(old_logp, np.float64))
    clipped = np.clip(ratio, 1.0 - eps, 1.0 + eps)
    s1, s2 = ratio * adv, clipped * adv
    l_clip = np.minimum(s1, s2).mean()
    ent = -(p * logp_all).sum(axis=1)
    # d min(s1, s2) / d logp: the unclipped branch is active when s1 <= s2 (ties go to it); the clipped one is flat
    active = s1 <= s2
    dlogp = np.where(active, ratio * adv, 0.0)
    onehot = np.zeros((B, A), np.float64)
    onehot[np.arange(B), a] = 1.0
    d_lclip = dlogp[:, None] * (onehot - p)                        # d logp_a / d z = onehot - p
    d_ent = -p * (logp_all + ent[:, None])                         # dH/dz_j = -p_j (log p_j + H)
    dlogits = -(d_lclip + beta * d_ent) / B
    v = np.asarray(values, np.float64)
    R = np.asarray(returns, np.float64)
    return {"l_clip": l_clip, "entropy": ent.mean(), "policy_loss": -(l_clip + beta * ent.mean()),
            "value_loss": (0.5 * (v - R) ** 2).mean(), "ratio": ratio, "dlogits": dlogits, "dvalues": (v - R) / B}
