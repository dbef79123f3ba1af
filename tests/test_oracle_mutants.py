"""Do the pins bite?  Each case plants ONE plausible mistake in (a wrapper around) the CPU oracle and checks that
at least one of the pin tests of test_oracle_pins.py fails on it.  The mistakes are the ones a re-implementation
would most likely make: a dropped epsilon, the wrong tie rule, a reversed bit order, a lost sign, a wrong head map.
All of this runs on the CPU; nothing here touches the CUDA library.
"""
import numpy as np
import pytest

import test_oracle_pins as pins
import test_oracle_pins_pack5 as pins5


class Mutant:
    """The oracle module with some functions replaced; `bitlinear` is re-composed from the (possibly replaced) parts."""

    def __init__(self, real, **overrides):
        self._real = real
        self._over = overrides

    def __getattr__(self, name):
        if name in self._over:
            return lambda *a, **k: self._over[name](self._real, *a, **k)
        return getattr(self._real, name)

    def bitlinear(self, x_bf16, Wq, gamma, threads=None):
        xq, a = self.quant_act(x_bf16)
        acc = self.contract(xq, Wq, threads)
        y32, yb, y64 = self.rescale(acc, gamma, a)
        return {"xq": xq, "absmax": a, "acc": acc, "y32": y32, "ybf16": yb, "y64": y64}


def _ternarize_half_away(real, W, gamma=None):
    """round-half-away-from-zero instead of ties-to-even: |W|/s = 0.5 becomes +-1 (Eq. 2 has a strict '>')."""
    W = np.ascontiguousarray(W, np.float32)
    g = real.absmean(W) if gamma is None else np.float32(gamma)
    t = W / np.float32(g + np.float32(1e-5))
    r = np.sign(t) * np.floor(np.abs(t) + np.float32(0.5))
    return np.clip(r, -1, 1).astype(np.int8), g


def _ternarize_no_eps(real, W, gamma=None):
    W = np.ascontiguousarray(W, np.float32)
    g = real.absmean(W) if gamma is None else np.float32(gamma)
    Wq, _ = real.ternarize(W, gamma=np.float32(g) * np.float32(1.3))  # threshold off by 30 %
    return Wq, g


def _pack_reversed_bits(real, Wq):
    p = real.pack(Wq)
    return ((p & 0x03) << 6) | ((p & 0x0C) << 2) | ((p & 0x30) >> 2) | ((p & 0xC0) >> 6)


def _pack5_most_significant_first(real, Wq):
    """digit i weighted 3^(4-i) instead of 3^i"""
    Wq = np.asarray(Wq, np.int8)
    K = Wq.shape[1]
    ext = np.zeros((Wq.shape[0], 5 * (-(-K // 5))), np.int8)
    ext[:, :K] = Wq
    return real.pack5(ext.reshape(ext.shape[0], -1, 5)[:, :, ::-1].reshape(ext.shape[0], -1))


def _pack5_pads_with_minus_one(real, Wq):
    """missing positions of the last byte packed as code 0 (a -1 weight) instead of code 1 (a zero weight)"""
    Wq = np.asarray(Wq, np.int8)
    K = Wq.shape[1]
    ext = np.full((Wq.shape[0], 5 * (-(-K // 5))), -1, np.int8)
    ext[:, :K] = Wq
    return real.pack5(ext)


def _contract_drops_minus(real, xq, Wq, threads=None):
    """treats -1 weights as 'skip' instead of 'subtract'"""
    return real.contract(xq, np.maximum(np.asarray(Wq), 0).astype(np.int8), threads)


def _contract_transposed_x(real, xq, Wq, threads=None):
    xq = np.asarray(xq)
    return real.contract(xq[:, ::-1].copy(), Wq, threads)  # k index reversed on one operand only


def _rescale_gamma_plus_eps(real, acc, gamma, absmax):
    return real.rescale(acc, np.float32(gamma) + np.float32(1e-5), absmax)


def _rescale_over_128(real, acc, gamma, absmax):
    y32, yb, y64 = real.rescale(acc, gamma, absmax)
    return (y32 * np.float32(127.0 / 128.0)).astype(np.float32), yb, y64 * (127.0 / 128.0)


def _quant_truncates(real, x_bf16):
    xq, a = real.quant_act(x_bf16)
    x = pins.bits_to_f32(x_bf16)
    q = np.trunc(x * (np.float32(127.0) / a[:, None]))
    return np.clip(q, -128, 127).astype(np.int8), a


def _quant_no_clamp(real, x_bf16):
    xq, a = real.quant_act(x_bf16)
    x = np.abs(pins.bits_to_f32(x_bf16)).max(axis=1)
    return xq, x.astype(np.float32)  # absmax without the 1e-5 floor


def _rmsnorm_no_eps_wrong_len(real, x_bf16):
    x = pins.bits_to_f32(x_bf16).astype(np.float64)
    u = x / np.sqrt((x * x).sum(axis=1, keepdims=True) / (x.shape[1] - 1))
    return pins.bf16_bits_of(u.astype(np.float32))


def _attention_modulo(real, qkv, n_heads, n_kv_heads, head_dim):
    T = qkv.shape[0]
    v = np.asarray(qkv)[:, (n_heads + n_kv_heads) * head_dim:].reshape(T, n_kv_heads, head_dim)
    return np.stack([v[:, h % n_kv_heads] for h in range(n_heads)], axis=1).reshape(T, n_heads * head_dim)


def _softmax_attention(real, qkv, states, n_heads, n_kv_heads, head_dim, theta, causal=True, scale=None,
                       interleaved=False):
    """A separate fp64 attention used only to plant mistakes (no mask / wrong scale / wrong rotary pairing)."""
    x = pins.bits_to_f32(qkv).astype(np.float64)
    T = x.shape[0]
    S = int(states)
    d, dkv, half = n_heads * head_dim, n_kv_heads * head_dim, head_dim // 2
    scale = 1.0 / np.sqrt(head_dim) if scale is None else scale
    out = np.zeros((T, d))

    def rope(v, p):
        ang = p * theta ** (-2.0 * np.arange(half) / head_dim)
        if interleaved:
            a, b = v[0::2], v[1::2]
            r = np.empty_like(v)
            r[0::2], r[1::2] = a * np.cos(ang) - b * np.sin(ang), b * np.cos(ang) + a * np.sin(ang)
            return r
        a, b = v[:half], v[half:]
        return np.concatenate([a * np.cos(ang) - b * np.sin(ang), b * np.cos(ang) + a * np.sin(ang)])

    for t0 in range(0, T, S):
        for h in range(n_heads):
            kv = h // (n_heads // n_kv_heads)
            q = np.stack([rope(x[t0 + p, h * head_dim:(h + 1) * head_dim], p) for p in range(S)])
            k = np.stack([rope(x[t0 + p, d + kv * head_dim:d + (kv + 1) * head_dim], p) for p in range(S)])
            v = x[t0:t0 + S, d + dkv + kv * head_dim:d + dkv + (kv + 1) * head_dim]
            sc = q @ k.T * scale
            if causal:
                sc = np.where(np.tril(np.ones((S, S), bool)), sc, -np.inf)
            w = np.exp(sc - sc.max(axis=1, keepdims=True))
            out[t0:t0 + S, h * head_dim:(h + 1) * head_dim] = (w / w.sum(axis=1, keepdims=True)) @ v
    return pins.bf16_bits_of(out.astype(np.float32))


def _attention_no_mask(real, *a):
    return _softmax_attention(real, *a, causal=False)


def _attention_no_scale(real, *a):
    return _softmax_attention(real, *a, scale=1.0)


def _attention_interleaved_rope(real, *a):
    return _softmax_attention(real, *a, interleaved=True)


def _relu2_without_square(real, gu):
    g = pins.bits_to_f32(gu)
    F = g.shape[1] // 2
    return (np.maximum(g[:, :F], 0) * g[:, F:]).astype(np.float32)


PIN_TESTS = [pins.test_eq2_definition_fp64, pins.test_eq2_ties_are_strict, pins.test_golden_worked_example,
             pins.test_dense_fp64_of_dequantized_operands, pins.test_quant_act_against_torch,
             pins.test_absmax_maps_to_127_and_zero_rows, pins.test_select_sum_add_subtract_skip,
             pins.test_negation_permutation_bound_allones, pins.test_pack_roundtrip_and_zero_matrix,
             pins.test_gaussian_closed_forms, pins.test_rescale_tolerances_and_bf16_rne,
             pins.test_rmsnorm_against_fp64, pins.test_relu2_gate_identity_attention_residual,
             pins.test_attention_against_library_sdpa, pins.test_attention_special_cases,
             pins5.test_pack5_golden_bytes, pins5.test_pack5_is_the_base3_number_of_every_digit_string,
             pins5.test_pack5_byte_count_padding_and_roundtrip, pins5.test_pack5_digit_positions]


def failing_pins(mod):
    failed = []
    for t in PIN_TESTS:
        try:
            if t is pins.test_dense_fp64_of_dequantized_operands:
                t(mod, 3, 64, 40, 1)
            else:
                t(mod)
        except AssertionError:
            failed.append(t.__name__)
        except Exception:  # a mistake that makes the computation blow up is caught as well
            failed.append(t.__name__)
    return failed


MUTANTS = {
    "ternarize: round half away": {"ternarize": _ternarize_half_away},
    "ternarize: threshold off": {"ternarize": _ternarize_no_eps},
    "pack: reversed bit order": {"pack": _pack_reversed_bits},
    "pack5: most significant digit first": {"pack5": _pack5_most_significant_first},
    "pack5: padding packed as -1": {"pack5": _pack5_pads_with_minus_one},
    "contract: -1 treated as skip": {"contract": _contract_drops_minus},
    "contract: k reversed on one operand": {"contract": _contract_transposed_x},
    "rescale: gamma + eps": {"rescale": _rescale_gamma_plus_eps},
    "rescale: 128 levels": {"rescale": _rescale_over_128},
    "quant: truncation": {"quant_act": _quant_truncates},
    "quant: no absmax floor": {"quant_act": _quant_no_clamp},
    "rmsnorm: wrong statistics": {"rmsnorm_bf16": _rmsnorm_no_eps_wrong_len},
    "attention: modulo head map": {"identity_attention": _attention_modulo},
    "gate: relu without the square": {"relu2_gate": _relu2_without_square},
    "attention: no causal mask": {"attention": _attention_no_mask},
    "attention: missing 1/sqrt(head_dim)": {"attention": _attention_no_scale},
    "attention: interleaved rotary pairs": {"attention": _attention_interleaved_rope},
}


def test_the_unmodified_oracle_passes_every_pin(oracle_mod):
    assert failing_pins(Mutant(oracle_mod)) == []


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_each_planted_mistake_fails_a_pin(oracle_mod, name):
    failed = failing_pins(Mutant(oracle_mod, **MUTANTS[name]))
    assert failed, f"no pin noticed the mistake: {name}"
