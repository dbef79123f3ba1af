"""Pins for the CPU oracle: every check here is computed WITHOUT the oracle's own code path for the thing
being checked (fp64 numpy restatements of the definition, exhaustive enumeration, closed forms, a
hand-worked fixture, library routines, algebraic invariants), so that a dropped term, a wrong sign or
index, or a transposed operand inside the oracle fails at least one of them.

Paper anchors: Sec. III-A Eq. 2 (ternary quantizer), Sec. III-A last paragraph (integer arithmetic,
no floating multiply-accumulate), Sec. V edge-deployment paragraph (additions and subtractions).
"""
import itertools
import json
import math
import os

import numpy as np
import pytest
import torch

from paper_2604_24273_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "bitlinear_worked_example.json")


def bf16_bits_of(a):
    """fp32 numpy -> bf16 bit patterns through torch's converter (library routine, RNE)."""
    return inputs.bf16_bits(torch.from_numpy(np.asarray(a, np.float32)).to(torch.bfloat16))


def bits_to_f32(bits):
    return (np.asarray(bits, np.uint16).astype(np.uint32) << 16).view(np.float32)


# ------------------------------------------------------------------------------------------ Eq. 2

def test_eq2_definition_fp64(oracle_mod):
    """W_q != 0  <=>  |W| > tau with tau = (gamma+1e-5)/2, sign(W_q) = sign(W)  (Eq. 2)."""
    W = inputs.master_weights(384, 512, 11).numpy()
    Wq, g = oracle_mod.ternarize(W)
    assert set(np.unique(Wq)) <= {-1, 0, 1}
    s = float(np.float32(g) + np.float32(1e-5))
    tau = s / 2.0
    a = np.abs(W.astype(np.float64))
    near = np.abs(a - tau) <= 1e-6 * tau  # fp32 division may land either side within an ulp of the edge
    want = np.sign(W.astype(np.float64)) * (a > tau)
    assert np.array_equal(Wq[~near].astype(np.float64), want[~near])
    assert near.sum() < 5
    # gamma against an independent fp64 mean
    assert abs(float(g) - np.abs(W.astype(np.float64)).mean()) <= 6e-8 * float(g)


def test_eq2_ties_are_strict(oracle_mod):
    """At |W|/s = 0.5 exactly the strict inequality of Eq. 2 gives 0; 1.5 and 2.5 clip to +-1."""
    gamma = np.float32(0.25) - np.float32(1e-5)
    s = np.float32(gamma + np.float32(1e-5))
    assert s == np.float32(0.25)  # exact by Sterbenz-free construction: check it really is
    W = np.array([[0.125, -0.125, 0.375, -0.375, 0.625, -0.625, 0.1250001, 0.0]], np.float32)
    Wq, _ = oracle_mod.ternarize(W, gamma=gamma)
    assert Wq.tolist() == [[0, 0, 1, -1, 1, -1, 1, 0]]


def test_golden_worked_example(oracle_mod):
    G = json.load(open(GOLDEN))
    W = np.array(G["W"], np.float32)
    Wq, g = oracle_mod.ternarize(W)
    assert abs(float(g) - G["gamma"]) < 1e-7
    assert Wq.tolist() == G["W_q"]
    assert oracle_mod.pack(Wq).tolist() == G["packed"]
    assert oracle_mod.unpack(np.array(G["packed"], np.uint8), 8).tolist() == G["W_q"]
    x = bf16_bits_of(np.array(G["x"], np.float32))
    r = oracle_mod.bitlinear(x, Wq, g)
    assert r["xq"].tolist() == G["x_q"]
    assert r["absmax"].tolist() == G["absmax"]
    assert r["acc"].tolist() == G["acc"]
    np.testing.assert_allclose(r["y64"], np.array(G["y"]), rtol=2e-7)
    np.testing.assert_allclose(r["y32"], np.array(G["y"]), rtol=1e-6)
    xt = bf16_bits_of(np.array(G["x_ties"], np.float32))
    assert np.array_equal(bits_to_f32(xt), np.array(G["x_ties"], np.float32))  # all bf16-exact
    xq, a = oracle_mod.quant_act(xt)
    assert xq.tolist() == G["x_ties_q"] and a.tolist() == [127.0]


# --------------------------------------------------------------------------- brute force, tiny

@pytest.mark.parametrize("K", [4, 8])
def test_exhaustive_ternary_rows(oracle_mod, K):
    """All 3^K weight rows (K=4: 81, K=8: 6561) against an integer dot and an fp64 dense product."""
    rows = np.array(list(itertools.product([-1, 0, 1], repeat=K)), np.int8)
    rng = np.random.default_rng(K)
    xq = rng.integers(-127, 128, size=(3, K)).astype(np.int8)
    acc = oracle_mod.contract(xq, rows, threads=2)
    want = xq.astype(np.int64) @ rows.astype(np.int64).T
    assert np.array_equal(acc.astype(np.int64), want)
    # pack / unpack on every pattern
    p = oracle_mod.pack(rows)
    assert np.array_equal(oracle_mod.unpack(p, K), rows)
    assert ((p >> 0) & 3).max() <= 2 and ((p >> 2) & 3).max() <= 2 and ((p >> 4) & 3).max() <= 2 \
        and ((p >> 6) & 3).max() <= 2
    # canonical bit positions restated: code of k in bits 2(k%4) of byte k//4
    for k in range(K):
        assert np.array_equal(((p[:, k // 4] >> (2 * (k % 4))) & 3).astype(np.int8) - 1, rows[:, k])


@pytest.mark.parametrize("M,K,N,seed", [(1, 16, 8, 0), (3, 64, 40, 1), (4, 32, 64, 2)])
def test_dense_fp64_of_dequantized_operands(oracle_mod, M, K, N, seed):
    """y64 equals the dense fp64 matmul (x_q*a/127) @ (gamma*W_q)^T; N != K catches a transposed operand."""
    W = inputs.master_weights(N, K, 100 + seed).numpy()
    x = inputs.activations(M, K, 200 + seed, outliers=False)
    Wq, g = oracle_mod.ternarize(W)
    r = oracle_mod.bitlinear(inputs.bf16_bits(x), Wq, g, threads=1)
    xd = r["xq"].astype(np.float64) * (r["absmax"].astype(np.float64)[:, None] / 127.0)
    wd = float(g) * Wq.astype(np.float64)
    dense = xd @ wd.T
    np.testing.assert_allclose(r["y64"], dense, rtol=1e-12, atol=1e-300)
    np.testing.assert_allclose(r["y32"], dense, rtol=1e-6, atol=0)
    # third opinion: torch integer matmul of the unpacked integers
    t = torch.from_numpy(r["xq"].astype(np.int32)) @ torch.from_numpy(Wq.astype(np.int32)).T
    assert np.array_equal(t.numpy(), r["acc"])


def test_contract_pairs_matches_full(oracle_mod):
    rng = np.random.default_rng(5)
    xq = rng.integers(-127, 128, size=(6, 128)).astype(np.int8)
    Wq = rng.integers(-1, 2, size=(20, 128)).astype(np.int8)
    want = xq.astype(np.int64) @ Wq.astype(np.int64).T
    ms, ns = np.meshgrid(np.arange(6), np.arange(20), indexing="ij")
    got = oracle_mod.contract_pairs(xq, Wq, ms.ravel(), ns.ravel())
    assert np.array_equal(got.astype(np.int64), want.ravel())


# -------------------------------------------------------------------------- act quant vs library

def test_quant_act_against_torch(oracle_mod):
    x = inputs.activations(5, 384, 7)
    xq, a = oracle_mod.quant_act(inputs.bf16_bits(x))
    xf = x.float()
    a_t = xf.abs().amax(dim=1).clamp_min(1e-5)
    inv = (torch.tensor(127.0) / a_t)[:, None]
    q_t = torch.clamp(torch.round(xf * inv), -128, 127).to(torch.int8)  # torch.round is half-to-even
    assert np.array_equal(a, a_t.numpy())
    assert np.array_equal(xq, q_t.numpy())


def test_absmax_maps_to_127_and_zero_rows(oracle_mod):
    x = inputs.activations(16, 256, 9)
    xb = inputs.bf16_bits(x)
    xq, a = oracle_mod.quant_act(xb)
    xf = x.float().numpy()
    for m in range(16):
        k = int(np.argmax(np.abs(xf[m])))
        assert abs(int(xq[m, k])) == 127 and np.sign(xq[m, k]) == np.sign(xf[m, k])
        assert np.abs(xq[m].astype(int)).max() == 127
    z = np.zeros((2, 64), np.uint16)
    zq, za = oracle_mod.quant_act(z)
    assert not zq.any() and np.all(za == np.float32(1e-5))


def test_power_of_two_scaling(oracle_mod):
    x = inputs.activations(4, 128, 10)
    W = inputs.master_weights(32, 128, 12).numpy()
    Wq, g = oracle_mod.ternarize(W)
    r1 = oracle_mod.bitlinear(inputs.bf16_bits(x), Wq, g)
    r2 = oracle_mod.bitlinear(inputs.bf16_bits((x.float() * 8.0).to(torch.bfloat16)), Wq, g)
    assert np.array_equal(r1["xq"], r2["xq"]) and np.array_equal(r1["acc"], r2["acc"])
    assert np.array_equal(r1["y32"] * np.float32(8.0), r2["y32"])


# ------------------------------------------------------------------------ contraction invariants

def _setup(oracle_mod, M=5, K=256, N=48, seed=3):
    W = inputs.master_weights(N, K, 300 + seed).numpy()
    x = inputs.activations(M, K, 400 + seed)
    Wq, g = oracle_mod.ternarize(W)
    xq, a = oracle_mod.quant_act(inputs.bf16_bits(x))
    return W, x, Wq, g, xq, a


def test_select_sum_add_subtract_skip(oracle_mod):
    """Each ternary dot product = sum of +1-selected activations minus sum of -1-selected ones (Sec. V)."""
    _, _, Wq, _, xq, _ = _setup(oracle_mod)
    acc = oracle_mod.contract(xq, Wq)
    for m in range(xq.shape[0]):
        for n in range(Wq.shape[0]):
            plus = int(xq[m][Wq[n] == 1].astype(np.int64).sum())
            minus = int(xq[m][Wq[n] == -1].astype(np.int64).sum())
            assert acc[m, n] == plus - minus


def test_zero_weights_contribute_nothing(oracle_mod):
    _, _, Wq, _, xq, _ = _setup(oracle_mod)
    acc = oracle_mod.contract(xq, Wq)
    rng = np.random.default_rng(0)
    for n in range(0, Wq.shape[0], 7):
        x2 = xq.copy()
        x2[:, Wq[n] == 0] = rng.integers(-127, 128, size=(xq.shape[0], int((Wq[n] == 0).sum())))
        acc2 = oracle_mod.contract(x2, Wq[n:n + 1])
        assert np.array_equal(acc2[:, 0], acc[:, n])


def test_negation_permutation_bound_allones(oracle_mod):
    W, x, Wq, g, xq, a = _setup(oracle_mod)
    acc = oracle_mod.contract(xq, Wq)
    # W -> -W and x -> -x negate exactly (round-to-nearest-even is odd-symmetric)
    Wq_n, g_n = oracle_mod.ternarize(-W)
    assert g_n == g and np.array_equal(Wq_n, -Wq)
    xq_n, a_n = oracle_mod.quant_act(inputs.bf16_bits(-x))
    assert np.array_equal(xq_n, -xq) and np.array_equal(a_n, a)
    assert np.array_equal(oracle_mod.contract(xq_n, Wq), -acc)
    # joint permutation of K
    perm = np.random.default_rng(1).permutation(xq.shape[1])
    assert np.array_equal(oracle_mod.contract(xq[:, perm], Wq[:, perm]), acc)
    # |acc| <= 127 * nnz
    nnz = (Wq != 0).sum(axis=1)
    assert np.all(np.abs(acc) <= 127 * nnz[None, :])
    # all +1 weights -> row sum of x_q
    ones = np.ones((3, xq.shape[1]), np.int8)
    assert np.array_equal(oracle_mod.contract(xq, ones), np.repeat(xq.astype(np.int64).sum(1)[:, None], 3, 1))


def test_row_independence(oracle_mod):
    """Quantization is per token: row m alone gives the same integers as row m inside a batch."""
    _, x, Wq, g, _, _ = _setup(oracle_mod, M=6)
    full = oracle_mod.bitlinear(inputs.bf16_bits(x), Wq, g)
    for m in (0, 3, 5):
        one = oracle_mod.bitlinear(inputs.bf16_bits(x[m:m + 1]), Wq, g)
        assert np.array_equal(one["xq"][0], full["xq"][m]) and np.array_equal(one["acc"][0], full["acc"][m])
        assert np.array_equal(one["ybf16"][0], full["ybf16"][m])


def test_pack_roundtrip_and_zero_matrix(oracle_mod):
    rng = np.random.default_rng(2)
    Wq = rng.integers(-1, 2, size=(37, 132)).astype(np.int8)
    p = oracle_mod.pack(Wq)
    assert p.shape == (37, 33) and np.array_equal(oracle_mod.unpack(p, 132), Wq)
    # no code 3 anywhere
    for s in (0, 2, 4, 6):
        assert ((p >> s) & 3).max() <= 2
    Z = np.zeros((4, 16), np.float32)
    Zq, gz = oracle_mod.ternarize(Z)
    assert gz == 0 and not Zq.any() and np.all(oracle_mod.pack(Zq) == 0x55)
    # packed size is exactly N*K/4 bytes = 1/8 of fp16 storage
    assert p.nbytes * 8 == Wq.size * 2


# --------------------------------------------------------------------------------- closed forms

def test_gaussian_closed_forms(oracle_mod):
    """N(0, sigma) weights: gamma -> sigma*sqrt(2/pi); P(W_q = 0) -> erf(tau/(sigma*sqrt 2))."""
    sigma = inputs.SIGMA_W
    W = inputs.master_weights(2560, 2560, 1001).numpy()
    Wq, g = oracle_mod.ternarize(W)
    g_cf = sigma * math.sqrt(2.0 / math.pi)
    assert abs(float(g) - g_cf) / g_cf < 1.5e-3
    tau = (g_cf + 1e-5) / 2.0
    p0 = math.erf(tau / (sigma * math.sqrt(2.0)))
    assert abs(p0 - 0.31025) < 3e-4  # the value quoted for "about one third zeros"
    assert abs(float((Wq == 0).mean()) - p0) < 1e-3
    assert abs(float((Wq == 1).mean()) - (1 - p0) / 2) < 1e-3
    assert abs(float((Wq == -1).mean()) - (1 - p0) / 2) < 1e-3


# -------------------------------------------------------------------------------------- rescale

def test_rescale_tolerances_and_bf16_rne(oracle_mod):
    W, x, Wq, g, xq, a = _setup(oracle_mod, M=7, K=512, N=96, seed=8)
    acc = oracle_mod.contract(xq, Wq)
    y32, yb, y64 = oracle_mod.rescale(acc, g, a)
    want = acc.astype(np.float64) * float(g) * a.astype(np.float64)[:, None] / 127.0
    np.testing.assert_allclose(y64, want, rtol=1e-15)
    nz = want != 0
    assert np.all(y32[~nz] == 0)
    assert np.max(np.abs(y32[nz] - want[nz]) / np.abs(want[nz])) < 4e-7
    yb_f = bits_to_f32(yb).astype(np.float64)
    assert np.max(np.abs(yb_f[nz] - want[nz]) / np.abs(want[nz])) < 2.0 ** -8 + 1e-6
    # the oracle's fp32 -> bf16 rounding equals the library converter (ties to even)
    assert np.array_equal(yb, bf16_bits_of(y32))
    # rescale uses gamma, not gamma + eps: with acc = 127 and a = 1, y = gamma exactly
    y1, _, _ = oracle_mod.rescale(np.array([[127]], np.int32), np.float32(0.5), np.array([1.0], np.float32))
    assert abs(float(y1[0, 0]) - 0.5) < 1e-7


# ----------------------------------------------------------------------------------------- glue

def test_rmsnorm_against_fp64(oracle_mod):
    x = inputs.activations(9, 640, 21)
    u = bits_to_f32(oracle_mod.rmsnorm_bf16(inputs.bf16_bits(x))).astype(np.float64)
    xd = x.double().numpy()
    want = xd / np.sqrt((xd * xd).mean(axis=1, keepdims=True) + 1e-5)
    assert np.max(np.abs(u - want) / np.maximum(np.abs(want), 1e-30)) <= 2.0 ** -8
    # exact bf16 rounding of the fp64 value except for double-rounding ties: allow 1 ulp on < 0.1 %
    wb = bf16_bits_of(want.astype(np.float32))
    assert (wb != oracle_mod.rmsnorm_bf16(inputs.bf16_bits(x))).mean() < 1e-3
    # unit RMS afterwards
    assert np.allclose((u * u).mean(axis=1), 1.0, atol=5e-3)
    xf = x.float().numpy()
    assert np.array_equal(oracle_mod.rmsnorm_f32(xf), oracle_mod.rmsnorm_bf16(inputs.bf16_bits(x)))


def test_relu2_gate_identity_attention_residual(oracle_mod):
    T, F = 5, 48
    gu = inputs.activations(T, 2 * F, 31, outliers=False)
    f = oracle_mod.relu2_gate(inputs.bf16_bits(gu))
    g = gu.double().numpy()[:, :F]
    up = gu.double().numpy()[:, F:]
    want = np.maximum(g, 0.0) ** 2 * up
    np.testing.assert_allclose(f, want, rtol=2e-7, atol=0)
    assert np.all(f[g <= 0] == 0)
    # identity attention: 4 query heads, 2 kv heads, head_dim 8  ->  head hd reads kv head hd // 2
    nh, nkv, hd = 4, 2, 8
    qkv = inputs.bf16_bits(inputs.activations(T, (nh + 2 * nkv) * hd, 32, outliers=False))
    att = oracle_mod.identity_attention(qkv, nh, nkv, hd)
    v = qkv[:, (nh + nkv) * hd:].reshape(T, nkv, hd)
    want_att = np.stack([v[:, h // (nh // nkv)] for h in range(nh)], axis=1).reshape(T, nh * hd)
    assert np.array_equal(att, want_att)
    # residual: fp32 add of two bf16, rounded to bf16 by the library converter
    a = inputs.activations(T, 64, 33)
    b = inputs.activations(T, 64, 34)
    got = oracle_mod.residual_add(inputs.bf16_bits(a), inputs.bf16_bits(b))
    assert np.array_equal(got, inputs.bf16_bits((a.float() + b.float()).to(torch.bfloat16)))


def test_encoder_block_is_the_composition(oracle_mod):
    """The fused block function equals the step-by-step composition of the pinned pieces."""
    dims = {"d": 256, "d_ff": 384, "n_heads": 2, "n_kv_heads": 1, "n_layers": 1}
    T = 6
    Ws = inputs.encoder_layer_weights(0, seed=77, dims=dims)
    layer = [oracle_mod.ternarize(w.numpy()) for w in Ws]
    h0 = inputs.bf16_bits(inputs.activations(T, dims["d"], 78))
    got = oracle_mod.encoder_block(h0, dims["d_ff"], 2, 1, layer, threads=2)
    o = oracle_mod
    u = o.rmsnorm_bf16(h0)
    qkv = o.bitlinear(u, *layer[0])["ybf16"]
    att = o.identity_attention(qkv, 2, 1, 128)
    y = o.bitlinear(o.rmsnorm_bf16(att), *layer[1])["ybf16"]
    h = o.residual_add(h0, y)
    gu = o.bitlinear(o.rmsnorm_bf16(h), *layer[2])["ybf16"]
    f = o.relu2_gate(gu)
    y = o.bitlinear(o.rmsnorm_f32(f), *layer[3])["ybf16"]
    h = o.residual_add(h, y)
    assert np.array_equal(got, h)
    assert got.shape == (T, 256) and np.isfinite(bits_to_f32(got)).all()


# ------------------------------------------------------------------------- attention (survey's NEXT row f1)

def _rope_complex(x, pos, theta):
    """Independent formulation of the rotary embedding: the pair (x_i, x_{i+hd/2}) as a complex number times e^{i*angle}."""
    hd = x.shape[-1]
    half = hd // 2
    ang = pos[:, None] * theta ** (-2.0 * np.arange(half) / hd)[None, :]
    z = (x[..., :half] + 1j * x[..., half:]) * np.exp(1j * ang)
    return np.concatenate([z.real, z.imag], axis=-1)


def test_attention_against_library_sdpa(oracle_mod):
    nh, nkv, hd, S, ns, theta = 4, 2, 16, 7, 3, 500000.0
    qkv = inputs.activations(ns * S, (nh + 2 * nkv) * hd, 41, outliers=False)
    got = bits_to_f32(oracle_mod.attention(inputs.bf16_bits(qkv), S, nh, nkv, hd, theta)).astype(np.float64)
    x = qkv.double().numpy().reshape(ns, S, -1)
    d, dkv = nh * hd, nkv * hd
    pos = np.arange(S, dtype=np.float64)
    q = np.stack([_rope_complex(x[:, :, h * hd:(h + 1) * hd].reshape(ns * S, hd), np.tile(pos, ns), theta)
                  for h in range(nh)], 1).reshape(ns, S, nh, hd)
    k = np.stack([_rope_complex(x[:, :, d + h * hd:d + (h + 1) * hd].reshape(ns * S, hd), np.tile(pos, ns), theta)
                  for h in range(nkv)], 1).reshape(ns, S, nkv, hd)
    v = x[:, :, d + dkv:].reshape(ns, S, nkv, hd)
    rep = nh // nkv
    qt = torch.from_numpy(q).permute(0, 2, 1, 3)
    kt = torch.from_numpy(np.repeat(k, rep, axis=2)).permute(0, 2, 1, 3)
    vt = torch.from_numpy(np.repeat(v, rep, axis=2)).permute(0, 2, 1, 3)
    want = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, is_causal=True)
    want = want.permute(0, 2, 1, 3).reshape(ns * S, nh * hd).numpy()
    assert np.max(np.abs(got - want) / np.maximum(np.abs(want), 1e-2)) <= 2.0 ** -8


def test_attention_special_cases(oracle_mod):
    nh, nkv, hd, theta = 4, 2, 16, 10000.0
    W = (nh + 2 * nkv) * hd
    d, dkv = nh * hd, nkv * hd
    # one token per state: the softmax is 1 and the output is V - exactly the "identity on V" block of the benchmark
    qkv1 = inputs.bf16_bits(inputs.activations(9, W, 42, outliers=False))
    assert np.array_equal(oracle_mod.attention(qkv1, 1, nh, nkv, hd, theta),
                          oracle_mod.identity_attention(qkv1, nh, nkv, hd))
    # q = 0: uniform causal weights, output = running mean of V
    S = 6
    x = inputs.activations(2 * S, W, 43, outliers=False).float().numpy()
    x[:, :d] = 0.0
    out = bits_to_f32(oracle_mod.attention(bf16_bits_of(x), S, nh, nkv, hd, theta)).astype(np.float64)
    xv = bits_to_f32(bf16_bits_of(x)).astype(np.float64)[:, d + dkv:].reshape(2, S, nkv, hd)
    run = np.cumsum(xv, axis=1) / np.arange(1, S + 1)[None, :, None, None]
    want = np.repeat(run, nh // nkv, axis=2).reshape(2 * S, d)
    assert np.max(np.abs(out - want)) <= 2.0 ** -8 * np.max(np.abs(want)) + 1e-6
    # causality: changing later tokens does not change earlier outputs; states do not see each other
    y = inputs.activations(2 * S, W, 44, outliers=False).float().numpy()
    base = oracle_mod.attention(bf16_bits_of(y), S, nh, nkv, hd, theta)
    y2 = y.copy()
    y2[4:6] += 1.0          # tokens 4, 5 of state 0
    pert = oracle_mod.attention(bf16_bits_of(y2), S, nh, nkv, hd, theta)
    assert np.array_equal(pert[:4], base[:4]) and np.array_equal(pert[S:], base[S:])
    assert not np.array_equal(pert[4:6], base[4:6])
    # constant V: every output equals that constant (weights sum to one)
    z = inputs.activations(S, W, 45, outliers=False).float().numpy()
    z[:, d + dkv:] = 0.75
    assert np.all(bits_to_f32(oracle_mod.attention(bf16_bits_of(z), S, nh, nkv, hd, theta)) == 0.75)


def test_attention_ragged_states_equal_separate_calls(oracle_mod):
    nh, nkv, hd, theta = 4, 2, 16, 500000.0
    lens = [3, 1, 8, 5]
    off = np.concatenate([[0], np.cumsum(lens)])
    qkv = inputs.bf16_bits(inputs.activations(int(off[-1]), (nh + 2 * nkv) * hd, 46, outliers=False))
    whole = oracle_mod.attention(qkv, off, nh, nkv, hd, theta)
    for s, n in enumerate(lens):
        part = oracle_mod.attention(qkv[off[s]:off[s + 1]], n, nh, nkv, hd, theta)
        assert np.array_equal(whole[off[s]:off[s + 1]], part)


def test_encoder_block_with_one_token_states_is_the_identity_attention_block(oracle_mod):
    """A state of one token attends to itself only, so the block with real attention reduces to the benchmark block."""
    d, d_ff, nh, nkv = 128, 256, 4, 2
    layer = []
    for j, (N, K) in enumerate([(d + 2 * nkv * (d // nh), d), (d, d), (2 * d_ff, d), (d, d_ff)]):
        layer.append(oracle_mod.ternarize(inputs.master_weights(N, K, 900 + j).numpy()))
    h = inputs.bf16_bits(inputs.activations(6, d, 47))
    a = oracle_mod.encoder_block(h, d_ff, nh, nkv, layer, threads=1)
    b = oracle_mod.encoder_block(h, d_ff, nh, nkv, layer, threads=1, states=1)
    c = oracle_mod.encoder_block(h, d_ff, nh, nkv, layer, threads=1, states=3)
    assert np.array_equal(a, b) and not np.array_equal(a, c)
    assert np.array_equal(a[[0, 3]], c[[0, 3]])   # the first token of each state sees only itself
