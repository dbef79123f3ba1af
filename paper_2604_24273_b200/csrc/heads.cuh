// The steps that follow the encoder: the trainable heads on the latent h_t (Eq. 3; Table VI: two hidden layers of 256
// and 128 units, fp32), generalized advantage estimation (Sec. III-B: lambda = 0.95, gamma = 0.99) and the clipped PPO
// objective (Eq. 1, eps = 0.1) with its entropy bonus (beta = 0.05).  All fp32; the batch is the parallel
// environments, every sample / environment is independent.
#pragma once

#include "common.cuh"

namespace bitrl {

constexpr int HEAD_MAX_HEADS = 4;
constexpr int HEAD_MAX_WIDTH = 256;  // hidden and output widths
constexpr int HEAD_KSPLIT = 4;       // the first layer's input range is split over four thread groups
constexpr int HEAD_THREADS = HEAD_MAX_WIDTH * HEAD_KSPLIT;

struct HeadsArgs {
  bitrl_head_t head[HEAD_MAX_HEADS];
  float* out[HEAD_MAX_HEADS];
  const unsigned short* h;  // bf16 [B, d]
  int B, d, H1, H2;
};

// out = tanh(tanh(h W1t + b1) W2t + b2) W3t + b3 for SB states per CTA; blockIdx.y = head.
// Layer 1 (d -> H1, nearly all of the work): thread (j, q) sums the q-th quarter of the inputs for output j and all SB
// states, reading W1t[k][j] coalesced over j; the quarters meet in shared memory.  Layers 2 and 3 are tiny.
template <int SB>
__global__ void __launch_bounds__(HEAD_THREADS) heads_forward_kernel(const __grid_constant__ HeadsArgs a) {
  extern __shared__ __align__(16) float hd_smem[];
  float* hs = hd_smem;                          // [SB][d]
  float* part = hs + SB * a.d;                  // [KSPLIT][SB][H1]
  float* a1 = part + HEAD_KSPLIT * SB * a.H1;   // [SB][H1]
  float* a2 = a1 + SB * a.H1;                   // [SB][H2]
  pdl_enter();
  const bitrl_head_t& hp = a.head[blockIdx.y];
  const int b0 = blockIdx.x * SB;
  const int nb = min(SB, a.B - b0);
  for (int i = threadIdx.x; i < SB * (a.d >> 1); i += HEAD_THREADS) {
    const int s = i / (a.d >> 1), k2 = i - s * (a.d >> 1);
    float lo = 0.0f, hi = 0.0f;
    if (s < nb) {
      const uint32_t raw = *reinterpret_cast<const uint32_t*>(a.h + static_cast<size_t>(b0 + s) * a.d + 2 * k2);
      lo = __uint_as_float(raw << 16);
      hi = __uint_as_float(raw & 0xffff0000u);
    }
    hs[s * a.d + 2 * k2] = lo;
    hs[s * a.d + 2 * k2 + 1] = hi;
  }
  __syncthreads();

  const int j = threadIdx.x % HEAD_MAX_WIDTH, q = threadIdx.x / HEAD_MAX_WIDTH;
  if (j < a.H1) {
    const int kq = a.d / HEAD_KSPLIT;  // d is a multiple of 16
    float acc[SB];
#pragma unroll
    for (int s = 0; s < SB; ++s) acc[s] = 0.0f;
    const float* w = hp.W1t + static_cast<size_t>(q) * kq * a.H1 + j;
    const float* x = hs + q * kq;
    // Every CTA reads the same weights: each starts at its own offset into the input range (and wraps), so that the
    // CTAs do not all ask the same L2 lines at the same moment.
    const int k_rot = static_cast<int>((blockIdx.x * 37u + blockIdx.y * 11u) % static_cast<unsigned>(kq / 4)) * 4;
#pragma unroll 1
    for (int pass = 0; pass < 2; ++pass) {
      const int k_lo = pass == 0 ? k_rot : 0, k_hi = pass == 0 ? kq : k_rot;
#pragma unroll(SB <= 4 ? 8 : 2)
      for (int k = k_lo; k < k_hi; k += 4) {
        const float w0 = w[static_cast<size_t>(k) * a.H1], w1 = w[static_cast<size_t>(k + 1) * a.H1],
                    w2 = w[static_cast<size_t>(k + 2) * a.H1], w3 = w[static_cast<size_t>(k + 3) * a.H1];
#pragma unroll
        for (int s = 0; s < SB; ++s) {
          const float4 xv = *reinterpret_cast<const float4*>(x + s * a.d + k);
          acc[s] = fmaf(xv.x, w0, acc[s]);
          acc[s] = fmaf(xv.y, w1, acc[s]);
          acc[s] = fmaf(xv.z, w2, acc[s]);
          acc[s] = fmaf(xv.w, w3, acc[s]);
        }
      }
    }
#pragma unroll
    for (int s = 0; s < SB; ++s) part[(q * SB + s) * a.H1 + j] = acc[s];
  }
  __syncthreads();
  for (int i = threadIdx.x; i < SB * a.H1; i += HEAD_THREADS) {
    const int s = i / a.H1, jj = i - s * a.H1;
    float v = hp.b1[jj];
#pragma unroll
    for (int qq = 0; qq < HEAD_KSPLIT; ++qq) v += part[(qq * SB + s) * a.H1 + jj];
    a1[i] = tanhf(v);
  }
  __syncthreads();
  for (int i = threadIdx.x; i < SB * a.H2; i += HEAD_THREADS) {
    const int s = i / a.H2, jj = i - s * a.H2;
    float v = hp.b2[jj];
    for (int k = 0; k < a.H1; ++k) v = fmaf(a1[s * a.H1 + k], hp.W2t[static_cast<size_t>(k) * a.H2 + jj], v);
    a2[i] = tanhf(v);
  }
  __syncthreads();
  const int O = hp.n_out;
  for (int i = threadIdx.x; i < SB * O; i += HEAD_THREADS) {
    const int s = i / O, jj = i - s * O;
    if (s >= nb) continue;
    float v = hp.b3[jj];
    for (int k = 0; k < a.H2; ++k) v = fmaf(a2[s * a.H2 + k], hp.W3t[static_cast<size_t>(k) * O + jj], v);
    a.out[blockIdx.y][static_cast<size_t>(b0 + s) * O + jj] = v;
  }
}

template <int SB>
bitrl_status launch_heads_t(const HeadsArgs& a, int n_heads, cudaStream_t st) {
  const size_t smem = sizeof(float) * (static_cast<size_t>(SB) * a.d + static_cast<size_t>(HEAD_KSPLIT + 1) * SB * a.H1 +
                                       static_cast<size_t>(SB) * a.H2);
  if (smem > 200 * 1024) return BITRL_ERR_SHAPE;
  BITRL_CUDA(cudaFuncSetAttribute(heads_forward_kernel<SB>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  static_cast<int>(smem)));
  BITRL_CUDA(launch_pdl(heads_forward_kernel<SB>, dim3((a.B + SB - 1) / SB, n_heads), dim3(HEAD_THREADS), smem, st, a));
  count_launch(1);
  return BITRL_OK;
}

bitrl_status launch_heads(const HeadsArgs& a, int n_heads, cudaStream_t st) {
  // few states: small tiles so that more SMs share the first layer's weights stream; many: larger tiles re-read it less
  if (a.B > 1024) return launch_heads_t<8>(a, n_heads, st);
  return a.B > 256 ? launch_heads_t<4>(a, n_heads, st) : launch_heads_t<2>(a, n_heads, st);
}

// GAE.  The recursion A_t = delta_t + c_t A_{t+1} (delta_t = r_t + gamma V_{t+1} (1 - done_t) - V_t, c_t = gamma lambda
// (1 - done_t)) is a chain of affine maps, and affine maps compose: a trajectory is cut into GAE_CHUNKS pieces, a thread
// folds its piece into A_first = Q + P * A_after (pass 1), one thread per environment chains the pieces from the end
// (pass 2), and every thread replays its piece with the now known A_after and writes the outputs (pass 3).  2048 steps
// become 3 x 64 dependent steps; the order of the fp32 operations differs from the plain backward loop only in how the
// pieces are joined.
constexpr int GAE_CHUNKS = 32;
constexpr int GAE_ENVS = 8;  // environments per CTA

__global__ void __launch_bounds__(GAE_CHUNKS * GAE_ENVS)
gae_kernel(const float* __restrict__ r, const float* __restrict__ v, const float* __restrict__ done, int T, int E,
           float gamma, float lam, float* __restrict__ adv, float* __restrict__ ret) {
  __shared__ float Ps[GAE_CHUNKS][GAE_ENVS], Qs[GAE_CHUNKS][GAE_ENVS], Ain[GAE_CHUNKS][GAE_ENVS];
  pdl_enter();
  const int el = threadIdx.x % GAE_ENVS, c = threadIdx.x / GAE_ENVS;
  const int e = blockIdx.x * GAE_ENVS + el;
  const bool live = e < E;
  const int len = (T + GAE_CHUNKS - 1) / GAE_CHUNKS;
  const int t_lo = c * len, t_hi = min(T, t_lo + len);  // this thread's steps [t_lo, t_hi)
  const float gl = __fmul_rn(gamma, lam);
  float P = 1.0f, Q = 0.0f;
  if (live) {
    for (int t = t_hi - 1; t >= t_lo; --t) {
      const size_t i = static_cast<size_t>(t) * E + e;
      const float nd = 1.0f - done[i];
      const float delta = r[i] + gamma * v[i + E] * nd - v[i];
      const float ct = gl * nd;
      Q = delta + ct * Q;
      P = ct * P;
    }
  }
  Ps[c][el] = P;
  Qs[c][el] = Q;
  __syncthreads();
  if (c == 0) {
    float a_after = 0.0f;  // A_T = 0
    for (int cc = GAE_CHUNKS - 1; cc >= 0; --cc) {
      Ain[cc][el] = a_after;
      a_after = Qs[cc][el] + Ps[cc][el] * a_after;
    }
  }
  __syncthreads();
  if (!live) return;
  float next_adv = Ain[c][el];
  for (int t = t_hi - 1; t >= t_lo; --t) {
    const size_t i = static_cast<size_t>(t) * E + e;
    const float nd = 1.0f - done[i], vt = v[i];
    const float delta = r[i] + gamma * v[i + E] * nd - vt;
    next_adv = delta + gl * nd * next_adv;
    adv[i] = next_adv;
    if (ret) ret[i] = next_adv + vt;
  }
}

// PPO objective, one warp per sample.  terms[b] = {ratio, min(r A, clip(r) A), entropy, 0.5 (V - R)^2}.
struct PpoArgs {
  const float* logits;  // [B, A]
  const int* actions;
  const float *old_logp, *adv, *values, *returns;
  int B, A;
  float eps, beta;
  float* terms;    // [B, 4]
  float* dlogits;  // [B, A] or null
  float* dvalues;  // [B] or null
};

__global__ void __launch_bounds__(256) ppo_terms_kernel(PpoArgs a) {
  pdl_enter();
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (b >= a.B) return;
  const float* z = a.logits + static_cast<size_t>(b) * a.A;
  float m = -INFINITY;
  for (int j = lane; j < a.A; j += 32) m = fmaxf(m, z[j]);
  m = warp_max(m);
  float se = 0.0f;
  for (int j = lane; j < a.A; j += 32) se += expf(z[j] - m);
  se = warp_sum(se);
  const float lse = logf(se);
  float ent = 0.0f;
  for (int j = lane; j < a.A; j += 32) {
    const float lp = z[j] - m - lse;
    ent -= expf(lp) * lp;
  }
  ent = warp_sum(ent);
  const int act = a.actions[b];
  const float logp = z[act] - m - lse;
  const float ratio = expf(logp - a.old_logp[b]);
  const float adv = a.adv[b];
  const float clipped = fminf(fmaxf(ratio, 1.0f - a.eps), 1.0f + a.eps);
  const float s1 = ratio * adv, s2 = clipped * adv;
  const float dv = a.values[b] - a.returns[b];
  if (lane == 0) {
    float4 t = make_float4(ratio, fminf(s1, s2), ent, 0.5f * dv * dv);
    *reinterpret_cast<float4*>(a.terms + 4 * static_cast<size_t>(b)) = t;
    if (a.dvalues) a.dvalues[b] = dv / static_cast<float>(a.B);
  }
  if (a.dlogits) {
    // d(-(L_clip + beta H))/dz_j = -( [s1 <= s2] r A (1[j = a] - p_j) - beta p_j (log p_j + H) ) / B
    const float dlogp = s1 <= s2 ? s1 : 0.0f;
    const float invB = 1.0f / static_cast<float>(a.B);
    float* dz = a.dlogits + static_cast<size_t>(b) * a.A;
    for (int j = lane; j < a.A; j += 32) {
      const float lp = z[j] - m - lse, p = expf(lp);
      const float g = dlogp * ((j == act ? 1.0f : 0.0f) - p) - a.beta * p * (lp + ent);
      dz[j] = -g * invB;
    }
  }
}

// Fixed-order sums over the batch: summary = {L_clip, mean entropy, -(L_clip + beta H), mean value error}.
__global__ void __launch_bounds__(256) ppo_summary_kernel(const float* terms, int B, float beta, float* summary) {
  __shared__ float red[3][256];
  pdl_enter();
  float s[3] = {0.0f, 0.0f, 0.0f};
  for (int b = threadIdx.x; b < B; b += 256) {
    const float4 t = *reinterpret_cast<const float4*>(terms + 4 * static_cast<size_t>(b));
    s[0] += t.y; s[1] += t.z; s[2] += t.w;
  }
  for (int c = 0; c < 3; ++c) red[c][threadIdx.x] = s[c];
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (threadIdx.x < o)
      for (int c = 0; c < 3; ++c) red[c][threadIdx.x] += red[c][threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const float invB = 1.0f / static_cast<float>(B);
    const float lc = red[0][0] * invB, en = red[1][0] * invB;
    summary[0] = lc;
    summary[1] = en;
    summary[2] = -(lc + beta * en);
    summary[3] = red[2][0] * invB;
  }
}

}  // namespace bitrl
