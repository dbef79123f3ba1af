"""GPU parity of the heads, GAE and PPO-objective kernels (through the C ABI) against the fp64 numpy oracle.

All three are fp32 on the GPU.  Tolerances, from the arithmetic:
  * heads: a d = 2560 fp32 dot product of O(1) terms carries ~sqrt(d) * 2^-24 * |terms| ~ 3e-6 absolute error, tanh is
    1-Lipschitz and the later layers are shorter: 2e-5 absolute on outputs of O(1) (plus 1e-5 relative).
  * GAE: the recursion's error is damped by gamma*lambda = 0.94 per step, so it stays at a few fp32 ulps of the
    running magnitude: 1e-5 relative to max|A| per environment.
  * PPO: exp/log in fp32 (2 ulp) on O(1) arguments: 1e-5 relative + 1e-6 absolute per sample; batch means 1e-5.
"""
import numpy as np
import pytest
import torch

from paper_2604_24273_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_24273_b200 import bitrl

    bitrl.lib()
    torch.cuda.set_device(0)
    return bitrl


def f64(t):
    return t.detach().cpu().to(torch.float64).numpy()


@pytest.mark.parametrize("nB,d,n_act", [(128, 2560, 6), (5, 2560, 2), (1030, 256, 17), (3, 64, 256)])
def test_heads_forward(oracle_mod, B, nB, d, n_act):
    h = inputs.activations(nB, d, 8100 + nB, outliers=False)
    pol = inputs.head_weights(d, n_act, 8200)
    val = inputs.head_weights(d, 1, 8201)
    logits, value = B.heads_forward(h.cuda(), [tuple(t.cuda() for t in pol), tuple(t.cuda() for t in val)])
    B.poll_status()
    want_l = oracle_mod.mlp_head(f64(h), *[f64(t) for t in pol])
    want_v = oracle_mod.mlp_head(f64(h), *[f64(t) for t in val])
    np.testing.assert_allclose(f64(logits), want_l, rtol=1e-5, atol=2e-5)
    np.testing.assert_allclose(f64(value), want_v, rtol=1e-5, atol=2e-5)


def test_heads_argument_errors(oracle_mod, B):
    h = inputs.activations(4, 64, 1, outliers=False).cuda()
    pol = tuple(t.cuda() for t in inputs.head_weights(64, 3, 2))
    descs = (B.HeadDesc * 1)(B.HeadDesc(*[t.data_ptr() for t in pol], 3))
    out = torch.empty((4, 3), dtype=torch.float32, device="cuda")
    optr = (B._vp * 1)(out.data_ptr())
    L = B.lib()
    assert L.bitrl_heads_forward(h.data_ptr(), 4, 60, 256, 128, descs, 1, optr, None) == B.ERR_SHAPE  # d % 16
    assert L.bitrl_heads_forward(h.data_ptr(), 4, 64, 512, 128, descs, 1, optr, None) == B.ERR_SHAPE  # H1 > 256
    assert L.bitrl_heads_forward(h.data_ptr(), 4, 64, 256, 128, descs, 5, optr, None) == B.ERR_SHAPE
    assert L.bitrl_heads_forward(None, 4, 64, 256, 128, descs, 1, optr, None) == B.ERR_NULL
    assert L.bitrl_heads_forward(h.data_ptr(), 4, 64, 256, 128, descs, 1, optr, None) == B.OK
    B.poll_status()


@pytest.mark.parametrize("T,E", [(2048, 128), (1, 1), (77, 300)])
def test_gae(oracle_mod, B, T, E):
    r, v, d = inputs.rollout(T, E, 8300 + T)
    adv, ret = B.gae(r.cuda(), v.cuda(), d.cuda(), 0.99, 0.95)
    B.poll_status()
    want_a, want_r = oracle_mod.gae(f64(r), f64(v), f64(d), 0.99, 0.95)
    scale = np.abs(want_a).max(axis=0, keepdims=True) + 1.0
    assert (np.abs(f64(adv) - want_a) <= 1e-5 * scale).all()
    assert (np.abs(f64(ret) - want_r) <= 1e-5 * (scale + np.abs(f64(v)[:T]))).all()


@pytest.mark.parametrize("nB,A", [(64, 6), (2048, 18), (7, 1), (33, 1000)])
def test_ppo_loss(oracle_mod, B, nB, A):
    logits, actions, old_logp, adv, v, R = inputs.ppo_batch(nB, A, 8400 + A)
    out = B.ppo_loss(*(t.cuda() for t in (logits, actions, old_logp, adv, v, R)), eps=0.1, beta=0.05)
    out2 = B.ppo_loss(*(t.cuda() for t in (logits, actions, old_logp, adv, v, R)), eps=0.1, beta=0.05)
    B.poll_status()
    want = oracle_mod.ppo_loss(f64(logits), actions.numpy(), f64(old_logp), f64(adv), f64(v), f64(R), 0.1, 0.05)
    s = f64(out["summary"])
    np.testing.assert_allclose(s, [want["l_clip"], want["entropy"], want["policy_loss"], want["value_loss"]],
                               rtol=1e-5, atol=1e-6)
    assert torch.equal(out["summary"], out2["summary"])  # fixed-order reduction: deterministic
    terms = f64(out["terms"])
    np.testing.assert_allclose(terms[:, 0], want["ratio"], rtol=1e-5)
    np.testing.assert_allclose(f64(out["dvalues"]), want["dvalues"], rtol=1e-6, atol=1e-9)
    # the gradient of a sample sitting exactly on the clip boundary is one-sided; none of the seeded samples does
    np.testing.assert_allclose(f64(out["dlogits"]), want["dlogits"], rtol=2e-5, atol=1e-6 / nB)


def test_gae_and_ppo_argument_errors(oracle_mod, B):
    L = B.lib()
    r, v, d = (t.cuda() for t in inputs.rollout(4, 3, 1))
    adv = torch.empty_like(r)
    assert L.bitrl_gae(r.data_ptr(), v.data_ptr(), d.data_ptr(), 0, 3, 0.99, 0.95, adv.data_ptr(), None, None) == B.ERR_SHAPE
    assert L.bitrl_gae(None, v.data_ptr(), d.data_ptr(), 4, 3, 0.99, 0.95, adv.data_ptr(), None, None) == B.ERR_NULL
    assert L.bitrl_gae(r.data_ptr(), v.data_ptr(), d.data_ptr(), 4, 3, 0.99, 0.95, adv.data_ptr(), None, None) == B.OK
    B.poll_status()
    want, _ = oracle_mod.gae(f64(r), f64(v), f64(d), 0.99, 0.95)  # returns pointer omitted: advantages only
    np.testing.assert_allclose(f64(adv), want, rtol=1e-5, atol=1e-5)
    logits, actions, old_logp, a_hat, val, R = (t.cuda() for t in inputs.ppo_batch(5, 4, 2))
    terms = torch.empty((5, 4), dtype=torch.float32, device="cuda")
    summ = torch.empty((4,), dtype=torch.float32, device="cuda")
    args = [logits.data_ptr(), actions.data_ptr(), old_logp.data_ptr(), a_hat.data_ptr(), val.data_ptr(), R.data_ptr()]
    assert L.bitrl_ppo_loss(*args, 0, 4, 0.1, 0.05, terms.data_ptr(), None, None, summ.data_ptr(), None) == B.ERR_SHAPE
    assert L.bitrl_ppo_loss(*args, 5, 4, 0.1, 0.05, None, None, None, summ.data_ptr(), None) == B.ERR_NULL
    assert L.bitrl_ppo_loss(*args, 5, 4, 0.1, 0.05, terms.data_ptr(), None, None, summ.data_ptr(), None) == B.OK  # no gradients asked
    B.poll_status()
    want = oracle_mod.ppo_loss(f64(logits), actions.cpu().numpy(), f64(old_logp), f64(a_hat), f64(val), f64(R), 0.1, 0.05)
    np.testing.assert_allclose(f64(summ), [want["l_clip"], want["entropy"], want["policy_loss"], want["value_loss"]],
                               rtol=1e-5, atol=1e-6)
