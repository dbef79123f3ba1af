// CPU oracle for the BitLinear W1.58A8 layer of the BitRL frozen backbone.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, obviously-correct statement of what the
// layer computes.  It shares no code with the CUDA library, is never called by the product path, and
// is only loaded by the tests, the smoke check and the benchmark's CPU-baseline leg.
//
// Every function is the definition written out as scalar loops (threads only split independent rows).
// fp32 steps are single IEEE operations, round-to-nearest-even, compiled with -ffp-contract=off so the
// compiler cannot fuse a multiply into an add.
//
// What the paper fixes and what it leaves open:
//   * Weights are ternary {-1,0,+1} (Abstract, Sec. I) produced by Q(W) = sign(W) * 1[|W| > tau]
//     (Sec. III-A, Eq. 2).  tau is not given; the reading used here is the absmean RoundClip quantizer of
//     the BitNet b1.58 layer the paper builds on: gamma = mean|W|, W_q = clip(round(W/(gamma+1e-5)),-1,1),
//     which is Eq. 2 with tau = (gamma+1e-5)/2 when "round" is ties-to-even.
//   * Inference is integer arithmetic without floating multiply-accumulate (Sec. III-A, last paragraph);
//     ternary products reduce to additions and subtractions (Sec. V, edge deployment paragraph).
//   * Activation quantization (int8, per-token absmax, Q = 127), the 2-bit packing and the rescale
//     gamma*absmax/127 are not in the paper; they are the W1.58A8 layer of the cited architecture.
//
// Pin status: every function below is pinned by tests that do not go through this file (fp64 dense
// matmul of dequantized operands, exhaustive tiny cases, closed forms for Gaussian weights, hand-worked
// fixtures, algebraic invariants).  No function is "parity unpinned".

#include <cmath>
#include <cstdint>
#include <cstring>
#include <thread>
#include <vector>
#include <algorithm>

namespace {

// bf16 <-> fp32.  bf16 is the upper 16 bits of an IEEE fp32.
inline float bf16_to_f32(uint16_t h) {
  uint32_t u = static_cast<uint32_t>(h) << 16;
  float f;
  std::memcpy(&f, &u, 4);
  return f;
}

// fp32 -> bf16, round to nearest, ties to even.  NaN stays NaN.
inline uint16_t f32_to_bf16_rne(float f) {
  uint32_t u;
  std::memcpy(&u, &f, 4);
  if ((u & 0x7fffffffu) > 0x7f800000u) return static_cast<uint16_t>((u >> 16) | 0x0040u);
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7fffu + lsb;
  return static_cast<uint16_t>(u >> 16);
}

template <class F>
void parallel_rows(int64_t rows, int threads, F f) {
  if (threads <= 1 || rows <= 1) {
    for (int64_t r = 0; r < rows; ++r) f(r);
    return;
  }
  int t = static_cast<int>(std::min<int64_t>(threads, rows));
  std::vector<std::thread> pool;
  for (int i = 0; i < t; ++i) {
    pool.emplace_back([=]() {
      for (int64_t r = i; r < rows; r += t) f(r);
    });
  }
  for (auto& th : pool) th.join();
}

}  // namespace

extern "C" {

// gamma = mean |W| over the whole matrix.  The sum is accumulated serially in fp64 (each fp32
// magnitude converts exactly) in row-major order and rounded to fp32 once.
float oracle_absmean(const float* W, int64_t count) {
  double S = 0.0;
  for (int64_t i = 0; i < count; ++i) S += std::fabs(static_cast<double>(W[i]));
  if (count == 0) return 0.0f;
  return static_cast<float>(S / static_cast<double>(count));
}

// Eq. 2 with tau = (gamma + 1e-5)/2, written as RoundClip:
//   s = gamma + 1e-5 (fp32 add), t = W/s (fp32 divide), r = rint(t) ties-to-even, W_q = clip(r,-1,1).
void oracle_ternarize(const float* W, int64_t count, float gamma, int8_t* Wq) {
  const float s = gamma + 1e-5f;
  for (int64_t i = 0; i < count; ++i) {
    float t = W[i] / s;
    float r = std::nearbyintf(t);  // default rounding mode = to nearest, ties to even
    if (r > 1.0f) r = 1.0f;
    if (r < -1.0f) r = -1.0f;
    Wq[i] = static_cast<int8_t>(r);
  }
}

// Canonical 2-bit packing: code c = W_q + 1 in {0,1,2}; byte j of row n holds k = 4j..4j+3, the code of
// k sits in bits [2(k mod 4)+1 : 2(k mod 4)].  Rows are contiguous, K/4 bytes each.  K % 4 == 0.
void oracle_pack(const int8_t* Wq, int64_t N, int64_t K, uint8_t* packed) {
  const int64_t KB = K / 4;
  for (int64_t n = 0; n < N; ++n) {
    for (int64_t j = 0; j < KB; ++j) {
      unsigned b = 0;
      for (int i = 0; i < 4; ++i) {
        unsigned c = static_cast<unsigned>(Wq[n * K + 4 * j + i] + 1);
        b |= (c & 3u) << (2 * i);
      }
      packed[n * KB + j] = static_cast<uint8_t>(b);
    }
  }
}

void oracle_unpack(const uint8_t* packed, int64_t N, int64_t K, int8_t* Wq) {
  const int64_t KB = K / 4;
  for (int64_t n = 0; n < N; ++n)
    for (int64_t k = 0; k < K; ++k) {
      unsigned b = packed[n * KB + k / 4];
      unsigned c = (b >> (2 * (k % 4))) & 3u;
      Wq[n * K + k] = static_cast<int8_t>(static_cast<int>(c) - 1);
    }
}

// Denser packing, five ternary weights per byte (1.6 bits per weight; the paper's "1.58-bit" weights of the Abstract
// and the lookup-table decoding of its inference stack, Sec. V edge-deployment paragraph).  The paper gives no format;
// the one used here is the base-3 number of the five codes c = W_q + 1:
//   byte j of row n = sum_{i=0..4} c[n, 5j+i] * 3^i      (0..242),   ceil(K/5) bytes per row,
// where positions 5j+i >= K (only in a row's last byte, when 5 does not divide K) count as W_q = 0, i.e. c = 1.
void oracle_pack5(const int8_t* Wq, int64_t N, int64_t K, uint8_t* packed) {
  const int64_t KB = (K + 4) / 5;
  for (int64_t n = 0; n < N; ++n) {
    for (int64_t j = 0; j < KB; ++j) {
      unsigned b = 0, p = 1;
      for (int i = 0; i < 5; ++i) {
        const int64_t k = 5 * j + i;
        const unsigned c = k < K ? static_cast<unsigned>(Wq[n * K + k] + 1) : 1u;
        b += c * p;
        p *= 3;
      }
      packed[n * KB + j] = static_cast<uint8_t>(b);
    }
  }
}

void oracle_unpack5(const uint8_t* packed, int64_t N, int64_t K, int8_t* Wq) {
  const int64_t KB = (K + 4) / 5;
  for (int64_t n = 0; n < N; ++n)
    for (int64_t k = 0; k < K; ++k) {
      unsigned b = packed[n * KB + k / 5];
      for (int i = 0; i < k % 5; ++i) b /= 3;
      Wq[n * K + k] = static_cast<int8_t>(static_cast<int>(b % 3) - 1);
    }
}

// Per-token absmax int8 quantization, Q = 127.  x is bf16 (raw 16-bit patterns), [M,K] row-major.
//   a = max_k |x|, a' = max(a, 1e-5), inv = 127/a' (fp32 divide), q = rint(x*inv) (one fp32 multiply,
//   ties-to-even), x_q = clip(q, -128, 127).
void oracle_quant_act(const uint16_t* x, int64_t M, int64_t K, int8_t* xq, float* absmax) {
  for (int64_t m = 0; m < M; ++m) {
    float a = 0.0f;
    for (int64_t k = 0; k < K; ++k) {
      float v = std::fabs(bf16_to_f32(x[m * K + k]));
      if (v > a) a = v;
    }
    if (a < 1e-5f) a = 1e-5f;
    const float inv = 127.0f / a;
    for (int64_t k = 0; k < K; ++k) {
      float q = std::nearbyintf(bf16_to_f32(x[m * K + k]) * inv);
      if (q > 127.0f) q = 127.0f;
      if (q < -128.0f) q = -128.0f;
      xq[m * K + k] = static_cast<int8_t>(q);
    }
    absmax[m] = a;
  }
}

// Eight-bit weights for the higher-precision critic backbone (Sec. V ablations, Table IV: "INT8 critic + 1-bit
// policy"; the paper names the precision only).  Reading: one symmetric absmax scale per matrix, the same rounding as
// the activations:  a = max(max|W|, 1e-20),  W_q = clip(rint(W * (127 / a)), -128, 127),  scale = a / 127.
// The layer then is the BitLinear formula with W_q in place of the ternary codes and `scale` in place of gamma:
//   acc = sum_k x_q W_q (int32, |acc| <= 127*128*K),  y = (float)acc * (scale * (a_m / 127)).
void oracle_w8_quantize(const float* W, int64_t count, int8_t* Wq, float* scale) {
  float a = 0.0f;
  for (int64_t i = 0; i < count; ++i) {
    const float v = std::fabs(W[i]);
    if (v > a) a = v;
  }
  if (a < 1e-20f) a = 1e-20f;
  const float inv = 127.0f / a;
  for (int64_t i = 0; i < count; ++i) {
    float q = std::nearbyintf(W[i] * inv);
    if (q > 127.0f) q = 127.0f;
    if (q < -128.0f) q = -128.0f;
    Wq[i] = static_cast<int8_t>(q);
  }
  *scale = a / 127.0f;
}

// Four-bit weights (the "INT4 critic" row of the same table), same reading with 7 in place of 127:
//   a = max(max|W|, 1e-20),  W_q = clip(rint(W * (7 / a)), -8, 7),  scale = a / 7.
// Codes are returned as int8 values in [-8, 7]; the layer is again the BitLinear formula with these codes and `scale`.
void oracle_w4_quantize(const float* W, int64_t count, int8_t* Wq, float* scale) {
  float a = 0.0f;
  for (int64_t i = 0; i < count; ++i) {
    const float v = std::fabs(W[i]);
    if (v > a) a = v;
  }
  if (a < 1e-20f) a = 1e-20f;
  const float inv = 7.0f / a;
  for (int64_t i = 0; i < count; ++i) {
    float q = std::nearbyintf(W[i] * inv);
    if (q > 7.0f) q = 7.0f;
    if (q < -8.0f) q = -8.0f;
    Wq[i] = static_cast<int8_t>(q);
  }
  *scale = a / 7.0f;
}

// Packed form of the four-bit codes: byte j of row n holds k = 2j (low nibble) and k = 2j+1 (high nibble), each as the
// biased code q + 8 in [0, 15].
void oracle_w4_pack(const int8_t* Wq, int64_t N, int64_t K, uint8_t* packed) {
  for (int64_t n = 0; n < N; ++n)
    for (int64_t j = 0; j < K / 2; ++j) {
      const unsigned lo = static_cast<unsigned>(Wq[n * K + 2 * j] + 8), hi = static_cast<unsigned>(Wq[n * K + 2 * j + 1] + 8);
      packed[n * (K / 2) + j] = static_cast<uint8_t>(lo | (hi << 4));
    }
}

// acc[m,n] = sum_k x_q[m,k] * W_q[n,k] in int32 (exact; |acc| <= 127*K for ternary, 127*128*K for 8-bit weights).
void oracle_contract(const int8_t* xq, const int8_t* Wq, int64_t M, int64_t N, int64_t K, int32_t* acc,
                     int threads) {
  parallel_rows(M, threads, [=](int64_t m) {
    for (int64_t n = 0; n < N; ++n) {
      int32_t s = 0;
      for (int64_t k = 0; k < K; ++k)
        s += static_cast<int32_t>(xq[m * K + k]) * static_cast<int32_t>(Wq[n * K + k]);
      acc[m * N + n] = s;
    }
  });
}

// The same contraction for a list of (m,n) pairs only; used to check full-size outputs one by one.
void oracle_contract_pairs(const int8_t* xq, const int8_t* Wq, int64_t K, const int64_t* ms,
                           const int64_t* ns, int64_t count, int32_t* acc) {
  for (int64_t i = 0; i < count; ++i) {
    int32_t s = 0;
    const int8_t* xr = xq + ms[i] * K;
    const int8_t* wr = Wq + ns[i] * K;
    for (int64_t k = 0; k < K; ++k) s += static_cast<int32_t>(xr[k]) * static_cast<int32_t>(wr[k]);
    acc[i] = s;
  }
}

// y = (float)acc * (gamma * (a'_m / 127)) in fp32, three single operations in this order.
// Any of y32 / ybf16 / y64 may be null.  y64 = (double)acc*gamma*a'/127 is the tolerance reference.
void oracle_rescale(const int32_t* acc, int64_t M, int64_t N, float gamma, const float* absmax, float* y32,
                    uint16_t* ybf16, double* y64) {
  for (int64_t m = 0; m < M; ++m) {
    const float t = absmax[m] / 127.0f;
    const float s = gamma * t;
    for (int64_t n = 0; n < N; ++n) {
      const float y = static_cast<float>(acc[m * N + n]) * s;
      if (y32) y32[m * N + n] = y;
      if (ybf16) ybf16[m * N + n] = f32_to_bf16_rne(y);
      if (y64)
        y64[m * N + n] = static_cast<double>(acc[m * N + n]) * static_cast<double>(gamma) *
                         static_cast<double>(absmax[m]) / 127.0;
    }
  }
}

// Whole layer on already-ternarized weights: quant -> contract -> rescale.  Optional taps may be null.
void oracle_bitlinear(const uint16_t* x, const int8_t* Wq, float gamma, int64_t M, int64_t N, int64_t K,
                      int8_t* xq_out, float* absmax_out, int32_t* acc_out, float* y32, uint16_t* ybf16,
                      double* y64, int threads) {
  std::vector<int8_t> xq_buf;
  std::vector<float> a_buf;
  std::vector<int32_t> acc_buf;
  int8_t* xq = xq_out;
  float* a = absmax_out;
  int32_t* acc = acc_out;
  if (!xq) { xq_buf.resize(static_cast<size_t>(M * K)); xq = xq_buf.data(); }
  if (!a) { a_buf.resize(static_cast<size_t>(M)); a = a_buf.data(); }
  if (!acc) { acc_buf.resize(static_cast<size_t>(M * N)); acc = acc_buf.data(); }
  oracle_quant_act(x, M, K, xq, a);
  oracle_contract(xq, Wq, M, N, K, acc, threads);
  oracle_rescale(acc, M, N, gamma, a, y32, ybf16, y64);
}

// ---------------------------------------------------------------------------------------------------
// Encoder glue (the paper only points to the BitNet papers for the block architecture, Sec. III-B; the
// readings are: gain 1, eps 1e-5, statistics in fp64, result rounded once to fp32 and then to bf16).

// u = x / sqrt(mean_k(x^2) + 1e-5), x given as fp32 [T,K]; output bf16.
void oracle_rmsnorm_f32(const float* x, int64_t T, int64_t K, uint16_t* u) {
  for (int64_t t = 0; t < T; ++t) {
    double ss = 0.0;
    for (int64_t k = 0; k < K; ++k) {
      double v = static_cast<double>(x[t * K + k]);
      ss += v * v;
    }
    const double r = 1.0 / std::sqrt(ss / static_cast<double>(K) + 1e-5);
    for (int64_t k = 0; k < K; ++k)
      u[t * K + k] = f32_to_bf16_rne(static_cast<float>(static_cast<double>(x[t * K + k]) * r));
  }
}

// The same with a bf16 input.
void oracle_rmsnorm_bf16(const uint16_t* x, int64_t T, int64_t K, uint16_t* u) {
  std::vector<float> row(static_cast<size_t>(K));
  for (int64_t t = 0; t < T; ++t) {
    for (int64_t k = 0; k < K; ++k) row[k] = bf16_to_f32(x[t * K + k]);
    oracle_rmsnorm_f32(row.data(), 1, K, u + t * K);
  }
}

// Gated FFN activation: f = max(g,0)^2 * up in fp32 (two single multiplies), g and up bf16.
// gu is [T, 2*F] with g = [:, 0:F] and up = [:, F:2F].  Output fp32 [T,F].
void oracle_relu2_gate(const uint16_t* gu, int64_t T, int64_t F, float* f) {
  for (int64_t t = 0; t < T; ++t)
    for (int64_t j = 0; j < F; ++j) {
      float g = bf16_to_f32(gu[t * 2 * F + j]);
      float up = bf16_to_f32(gu[t * 2 * F + F + j]);
      float r = g > 0.0f ? g : 0.0f;
      float r2 = r * r;
      f[t * F + j] = r2 * up;
    }
}

// "Identity attention": with one key per query the softmax is 1 and the head output is V.  With grouped
// KV heads, query head hd reads kv head hd / (n_heads / n_kv_heads).  qkv is bf16 [T, d + 2*dkv] with
// v = [:, d+dkv : d+2*dkv]; att is bf16 [T, d].
void oracle_identity_attention(const uint16_t* qkv, int64_t T, int64_t n_heads, int64_t n_kv_heads,
                               int64_t head_dim, uint16_t* att) {
  const int64_t d = n_heads * head_dim, dkv = n_kv_heads * head_dim, W = d + 2 * dkv;
  const int64_t rep = n_heads / n_kv_heads;
  for (int64_t t = 0; t < T; ++t)
    for (int64_t hd = 0; hd < n_heads; ++hd)
      for (int64_t e = 0; e < head_dim; ++e)
        att[t * d + hd * head_dim + e] = qkv[t * W + d + dkv + (hd / rep) * head_dim + e];
}

// Real attention inside each state (the step after the hot path; the paper only says that a state serializes to
// 15-40 tokens that the backbone processes in one forward pass, Sec. V, and that h_t = f(serialize(s_t)), Eq. 3; the
// form below is the causal grouped-query attention with rotary embedding of the cited architecture).
// qkv: bf16 [T, (n_heads + 2 n_kv_heads) * head_dim] = [q | k | v]; state s owns the contiguous tokens
// state_off[s] .. state_off[s+1]-1 (lengths may differ from state to state); T = state_off[n_states].
//   rotary (rotate-half form), position p = index of the token inside its state, for i < head_dim/2:
//     angle = p * theta^(-2 i / head_dim);  (x_i, x_{i+hd/2}) -> (x_i cos - x_{i+hd/2} sin, x_{i+hd/2} cos + x_i sin)
//   applied to q and k.  score(p, r) = q_p . k_r / sqrt(head_dim) for r <= p, softmax over r, out_p = sum_r w_r v_r.
// Query head h reads kv head h / (n_heads / n_kv_heads).  Everything in fp64; output rounded once to fp32, then bf16.
void oracle_attention(const uint16_t* qkv, const int64_t* state_off, int64_t n_states, int64_t n_heads,
                      int64_t n_kv_heads, int64_t head_dim, double theta, uint16_t* att) {
  const int64_t d = n_heads * head_dim, dkv = n_kv_heads * head_dim, W = d + 2 * dkv, half = head_dim / 2;
  const int64_t rep = n_heads / n_kv_heads;
  std::vector<double> q, k, w;
  auto rope = [&](const uint16_t* src, int64_t pos, double* dst) {
    for (int64_t i = 0; i < half; ++i) {
      const double ang = static_cast<double>(pos) * std::pow(theta, -2.0 * static_cast<double>(i) / static_cast<double>(head_dim));
      const double c = std::cos(ang), sn = std::sin(ang);
      const double a = bf16_to_f32(src[i]), b = bf16_to_f32(src[i + half]);
      dst[i] = a * c - b * sn;
      dst[i + half] = b * c + a * sn;
    }
  };
  for (int64_t st = 0; st < n_states; ++st) {
    const int64_t t0 = state_off[st], S = state_off[st + 1] - state_off[st];
    q.assign(static_cast<size_t>(S * head_dim), 0.0);
    k.assign(static_cast<size_t>(S * head_dim), 0.0);
    w.assign(static_cast<size_t>(S), 0.0);
    for (int64_t h = 0; h < n_heads; ++h) {
      const int64_t kvh = h / rep;
      for (int64_t p = 0; p < S; ++p) {
        const uint16_t* row = qkv + (t0 + p) * W;
        rope(row + h * head_dim, p, q.data() + p * head_dim);
        rope(row + d + kvh * head_dim, p, k.data() + p * head_dim);
      }
      for (int64_t p = 0; p < S; ++p) {
        double mx = -1e300;
        for (int64_t r = 0; r <= p; ++r) {
          double sc = 0.0;
          for (int64_t e = 0; e < head_dim; ++e) sc += q[p * head_dim + e] * k[r * head_dim + e];
          w[r] = sc / std::sqrt(static_cast<double>(head_dim));
          if (w[r] > mx) mx = w[r];
        }
        double den = 0.0;
        for (int64_t r = 0; r <= p; ++r) { w[r] = std::exp(w[r] - mx); den += w[r]; }
        for (int64_t e = 0; e < head_dim; ++e) {
          double o = 0.0;
          for (int64_t r = 0; r <= p; ++r)
            o += w[r] * static_cast<double>(bf16_to_f32(qkv[(t0 + r) * W + d + dkv + kvh * head_dim + e]));
          att[(t0 + p) * d + h * head_dim + e] = f32_to_bf16_rne(static_cast<float>(o / den));
        }
      }
    }
  }
}

// Residual: h <- bf16( fp32(h) + fp32(y) ), both bf16.
void oracle_residual_add(uint16_t* h, const uint16_t* y, int64_t count) {
  for (int64_t i = 0; i < count; ++i) h[i] = f32_to_bf16_rne(bf16_to_f32(h[i]) + bf16_to_f32(y[i]));
}

// One encoder block on a bf16 residual stream h [T,d], in place:
//   h += BitLinear_out( RMSNorm( identity_attention( BitLinear_qkv( RMSNorm(h) ) ) ) )
//   h += BitLinear_down( RMSNorm( relu2_gate( BitLinear_gateup( RMSNorm(h) ) ) ) )
// Wq_* are int8 ternary matrices [N,K] with scales g_*.  With state_off == nullptr the attention step is the
// identity on V above; otherwise it is oracle_attention over the states state_off describes (rotary base theta).
void oracle_encoder_block_states(uint16_t* h, int64_t T, int64_t d, int64_t d_ff, int64_t n_heads,
                                 int64_t n_kv_heads, const int8_t* Wq_qkv, float g_qkv, const int8_t* Wq_out,
                                 float g_out, const int8_t* Wq_gu, float g_gu, const int8_t* Wq_down, float g_down,
                                 const int64_t* state_off, int64_t n_states, double theta, int threads) {
  const int64_t head_dim = d / n_heads;
  const int64_t n_qkv = d + 2 * n_kv_heads * head_dim;
  std::vector<uint16_t> u(static_cast<size_t>(T * std::max(d, d_ff)));
  std::vector<uint16_t> qkv(static_cast<size_t>(T * n_qkv));
  std::vector<uint16_t> att(static_cast<size_t>(T * d));
  std::vector<uint16_t> y(static_cast<size_t>(T * d));
  std::vector<uint16_t> gu(static_cast<size_t>(T * 2 * d_ff));
  std::vector<float> f(static_cast<size_t>(T * d_ff));

  oracle_rmsnorm_bf16(h, T, d, u.data());
  oracle_bitlinear(u.data(), Wq_qkv, g_qkv, T, n_qkv, d, nullptr, nullptr, nullptr, nullptr, qkv.data(),
                   nullptr, threads);
  if (state_off)
    oracle_attention(qkv.data(), state_off, n_states, n_heads, n_kv_heads, head_dim, theta, att.data());
  else
    oracle_identity_attention(qkv.data(), T, n_heads, n_kv_heads, head_dim, att.data());
  oracle_rmsnorm_bf16(att.data(), T, d, u.data());
  oracle_bitlinear(u.data(), Wq_out, g_out, T, d, d, nullptr, nullptr, nullptr, nullptr, y.data(), nullptr,
                   threads);
  oracle_residual_add(h, y.data(), T * d);

  oracle_rmsnorm_bf16(h, T, d, u.data());
  oracle_bitlinear(u.data(), Wq_gu, g_gu, T, 2 * d_ff, d, nullptr, nullptr, nullptr, nullptr, gu.data(),
                   nullptr, threads);
  oracle_relu2_gate(gu.data(), T, d_ff, f.data());
  oracle_rmsnorm_f32(f.data(), T, d_ff, u.data());
  oracle_bitlinear(u.data(), Wq_down, g_down, T, d, d_ff, nullptr, nullptr, nullptr, nullptr, y.data(),
                   nullptr, threads);
  oracle_residual_add(h, y.data(), T * d);
}

void oracle_encoder_block(uint16_t* h, int64_t T, int64_t d, int64_t d_ff, int64_t n_heads,
                          int64_t n_kv_heads, const int8_t* Wq_qkv, float g_qkv, const int8_t* Wq_out,
                          float g_out, const int8_t* Wq_gu, float g_gu, const int8_t* Wq_down, float g_down,
                          int threads) {
  oracle_encoder_block_states(h, T, d, d_ff, n_heads, n_kv_heads, Wq_qkv, g_qkv, Wq_out, g_out, Wq_gu, g_gu, Wq_down,
                              g_down, nullptr, 0, 0.0, threads);
}

}  // extern "C"
