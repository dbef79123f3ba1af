"""Pins of the oracle's head / GAE / PPO functions against things other than the oracle itself: closed forms, brute
force written from the definitions, special cases, library routines (torch distributions, autograd, linear) and
finite differences.  Each planted mistake named in a test's docstring makes that test fail."""
import math

import numpy as np
import pytest
import torch

import oracle


def test_gae_lambda_one_is_discounted_return_minus_value():
    """lambda = 1 telescopes: A_t = sum_l gamma^l r_{t+l} + gamma^(T-t) V_T - V_t (brute-force double loop).
    Catches a wrong bootstrap index, a dropped gamma, a forward instead of backward recursion."""
    rng = np.random.default_rng(0)
    T, E, g = 17, 3, 0.9
    r, v = rng.normal(size=(T, E)), rng.normal(size=(T + 1, E))
    adv, ret = oracle.gae(r, v, np.zeros((T, E)), g, 1.0)
    for t in range(T):
        want = sum(g ** l * r[t + l] for l in range(T - t)) + g ** (T - t) * v[T] - v[t]
        np.testing.assert_allclose(adv[t], want, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(ret, adv + v[:T], rtol=0, atol=0)


def test_gae_lambda_zero_is_td_error_and_geometric_closed_form():
    rng = np.random.default_rng(1)
    T, E = 9, 2
    r, v = rng.normal(size=(T, E)), rng.normal(size=(T + 1, E))
    adv, _ = oracle.gae(r, v, np.zeros((T, E)), 0.99, 0.0)
    np.testing.assert_allclose(adv, r + 0.99 * v[1:] - v[:-1], rtol=1e-13)
    # constant reward, zero values: A_t = r (1 - c^(T-t)) / (1 - c), c = gamma * lambda
    adv, _ = oracle.gae(np.full((T, 1), 2.0), np.zeros((T + 1, 1)), np.zeros((T, 1)), 0.99, 0.95)
    c = 0.99 * 0.95
    want = np.array([2.0 * (1 - c ** (T - t)) / (1 - c) for t in range(T)])
    np.testing.assert_allclose(adv[:, 0], want, rtol=1e-12)


def test_gae_done_cuts_the_recursion_and_the_bootstrap():
    """After done_t = 1 neither V_{t+1} nor A_{t+1} reaches step t: the episode before the cut equals GAE run on it alone."""
    rng = np.random.default_rng(2)
    T = 12
    r, v = rng.normal(size=(T, 1)), rng.normal(size=(T + 1, 1))
    d = np.zeros((T, 1)); d[6] = 1.0
    adv, _ = oracle.gae(r, v, d, 0.99, 0.95)
    v_first = v[:8].copy(); v_first[7] = 0.0  # terminal: no bootstrap
    adv_first, _ = oracle.gae(r[:7], v_first, np.zeros((7, 1)), 0.99, 0.95)
    np.testing.assert_allclose(adv[:7], adv_first, rtol=1e-12)
    adv_second, _ = oracle.gae(r[7:], v[7:], np.zeros((T - 7, 1)), 0.99, 0.95)
    np.testing.assert_allclose(adv[7:], adv_second, rtol=1e-12)


def test_mlp_head_against_torch_linear_and_a_hand_case():
    rng = np.random.default_rng(3)
    B, d, H1, H2, O = 5, 24, 16, 8, 3
    h = rng.normal(size=(B, d)); W1t = rng.normal(size=(d, H1)) * 0.3; b1 = rng.normal(size=H1)
    W2t = rng.normal(size=(H1, H2)) * 0.3; b2 = rng.normal(size=H2); W3t = rng.normal(size=(H2, O)); b3 = rng.normal(size=O)
    got = oracle.mlp_head(h, W1t, b1, W2t, b2, W3t, b3)
    F = torch.nn.functional
    t = lambda a: torch.from_numpy(np.asarray(a, np.float64))
    x = torch.tanh(F.linear(t(h), t(W1t).T, t(b1)))
    x = torch.tanh(F.linear(x, t(W2t).T, t(b2)))
    want = F.linear(x, t(W3t).T, t(b3)).numpy()
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)
    # hand case: one input, one unit per layer: out = w3 * tanh(w2 * tanh(w1 * x + b1) + b2) + b3
    one = oracle.mlp_head([[0.5]], [[2.0]], [0.1], [[-1.5]], [0.2], [[3.0]], [-0.4])
    assert one.shape == (1, 1)
    assert abs(one[0, 0] - (3.0 * math.tanh(-1.5 * math.tanh(2.0 * 0.5 + 0.1) + 0.2) - 0.4)) < 1e-15


def _batch(seed, B=11, A=5):
    rng = np.random.default_rng(seed)
    logits = rng.normal(size=(B, A)) * 2
    actions = rng.integers(0, A, size=B)
    old_logp = oracle.log_softmax(logits + rng.normal(size=(B, A)) * 0.3)[np.arange(B), actions]
    return logits, actions, old_logp, rng.normal(size=B), rng.normal(size=B), rng.normal(size=B)


def test_ppo_special_cases_ratio_one_uniform_entropy_and_clip_branches():
    """ratio = 1 gives L_CLIP = mean(A); uniform logits have entropy log(A); a ratio above 1+eps with positive
    advantage contributes (1+eps) A and no gradient, below 1-eps with negative advantage (1-eps) A; the pessimistic
    min keeps the unclipped term when it is the smaller one.  Catches max instead of min, a clip on the wrong side,
    a missing sign on the entropy."""
    logits, actions, _, adv, v, R = _batch(4)
    B, A = logits.shape
    logp = oracle.log_softmax(logits)[np.arange(B), actions]
    out = oracle.ppo_loss(logits, actions, logp, adv, v, R)
    assert abs(out["l_clip"] - adv.mean()) < 1e-14 and np.allclose(out["ratio"], 1.0)
    out = oracle.ppo_loss(np.zeros((B, A)), actions, np.full(B, -math.log(A)), adv, v, R)
    assert abs(out["entropy"] - math.log(A)) < 1e-14
    # two actions, one sample, crafted ratios
    z = np.array([[0.0, 0.0]])
    for ratio, a_hat, want, grad_zero in [(1.5, 2.0, 1.1 * 2.0, True), (0.5, -2.0, 0.9 * -2.0, True),
                                          (1.5, -2.0, 1.5 * -2.0, False), (0.5, 2.0, 0.5 * 2.0, False)]:
        old = math.log(0.5) - math.log(ratio)
        out = oracle.ppo_loss(z, [0], [old], [a_hat], [0.0], [0.0], eps=0.1, beta=0.0)
        assert abs(out["l_clip"] - want) < 1e-14
        assert np.allclose(out["dlogits"], 0.0) == grad_zero


def test_ppo_terms_against_torch_distributions_and_autograd():
    """log-prob and entropy from torch.distributions.Categorical, gradients from autograd on torch's own min/clamp."""
    logits, actions, old_logp, adv, v, R = _batch(5)
    out = oracle.ppo_loss(logits, actions, old_logp, adv, v, R, eps=0.1, beta=0.05)
    z = torch.tensor(logits, dtype=torch.float64, requires_grad=True)
    vt = torch.tensor(v, dtype=torch.float64, requires_grad=True)
    dist = torch.distributions.Categorical(logits=z)
    ratio = torch.exp(dist.log_prob(torch.tensor(actions)) - torch.tensor(old_logp))
    A_hat = torch.tensor(adv)
    l_clip = torch.minimum(ratio * A_hat, torch.clamp(ratio, 0.9, 1.1) * A_hat).mean()
    ent = dist.entropy().mean()
    policy_loss = -(l_clip + 0.05 * ent)
    value_loss = (0.5 * (vt - torch.tensor(R)) ** 2).mean()
    policy_loss.backward(); value_loss.backward()
    assert abs(out["l_clip"] - l_clip.item()) < 1e-13 and abs(out["entropy"] - ent.item()) < 1e-13
    assert abs(out["policy_loss"] - policy_loss.item()) < 1e-13 and abs(out["value_loss"] - value_loss.item()) < 1e-13
    np.testing.assert_allclose(out["ratio"], ratio.detach().numpy(), rtol=1e-13)
    np.testing.assert_allclose(out["dlogits"], z.grad.numpy(), rtol=1e-10, atol=1e-14)
    np.testing.assert_allclose(out["dvalues"], vt.grad.numpy(), rtol=1e-12, atol=1e-15)


def test_ppo_gradient_against_finite_differences():
    logits, actions, old_logp, adv, v, R = _batch(6, B=4, A=3)
    out = oracle.ppo_loss(logits, actions, old_logp, adv, v, R)
    h = 1e-6
    for b in range(4):
        for j in range(3):
            zp, zm = logits.copy(), logits.copy()
            zp[b, j] += h; zm[b, j] -= h
            fd = (oracle.ppo_loss(zp, actions, old_logp, adv, v, R)["policy_loss"] -
                  oracle.ppo_loss(zm, actions, old_logp, adv, v, R)["policy_loss"]) / (2 * h)
            assert abs(fd - out["dlogits"][b, j]) < 1e-7


def test_log_softmax_normalizes_and_is_shift_invariant():
    rng = np.random.default_rng(7)
    z = rng.normal(size=(6, 9)) * 30
    lp = oracle.log_softmax(z)
    np.testing.assert_allclose(np.exp(lp).sum(1), 1.0, rtol=1e-13)
    np.testing.assert_allclose(oracle.log_softmax(z + 1000.0), lp, rtol=0, atol=1e-10)
    np.testing.assert_allclose(lp, torch.log_softmax(torch.tensor(z), dim=1).numpy(), rtol=1e-12, atol=1e-12)
