// Attention inside each state of the frozen encoder (Eq. 3: h_t = f(serialize(s_t)); Sec. V: a state serializes
// to 15-40 tokens that go through the backbone in one forward pass).  Causal grouped-query attention with rotary
// position embedding, the form of the architecture the backbone follows (Sec. III-B cites it, the paper does not
// spell it out).  States are short and independent, so one CTA owns one (state, kv head): its rotated keys and its
// values sit in shared memory as fp32 and every query of the heads that share the kv head streams over them.
//
//   rotary (rotate-half), position p = index of the token inside its state, i < head_dim/2:
//     angle = p * theta^(-2i/head_dim);  (x_i, x_{i+hd/2}) -> (x_i cos - x_{i+hd/2} sin, x_{i+hd/2} cos + x_i sin)
//   score(p, r) = q_p . k_r / sqrt(head_dim), r <= p;  w = exp(score - max);  out_p = (sum_r w_r v_r) / sum_r w_r
//
// All arithmetic is fp32 (fused multiply-adds), the cos/sin table is computed in fp64 and rounded once; the output
// is rounded once to bf16.  Also here: last-token pooling of the encoder output to one latent per state.
#pragma once

#include <cuda_fp16.h>

#include "common.cuh"

namespace bitrl {

constexpr int ATT_THREADS = 256;
constexpr int ATT_WARPS = ATT_THREADS / 32;
constexpr int ATT_STAGE_BAD_STATE = 120;  // stage id reported when a state's offsets are invalid

struct AttArgs {
  const unsigned short* qkv;  // bf16 [T, (n_heads + 2 n_kv) * HD] = [q | k | v]
  const int* state_off;       // device [n_states + 1], or nullptr for equal lengths
  int state_len;              // common length when state_off == nullptr; else the largest length allowed
  int T;
  int n_heads, n_kv;
  const float2* rope;         // [state_len][HD / 2]: (cos, sin) of position * theta^(-2i/HD)
  unsigned short* att;        // bf16 [T, n_heads * HD]
};

__device__ __forceinline__ uint32_t ptx_smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void report_status(int status, int stage) {
  if (atomicCAS(&g_status[0], 0, status) == 0) g_status[1] = stage;
}

// Token range of state `st`; false (and a status word) when the offsets do not describe 1..max_len tokens inside T.
__device__ __forceinline__ bool state_range(const int* state_off, int state_len, int T, int st, int& t0, int& S) {
  if (state_off) {
    t0 = state_off[st];
    S = state_off[st + 1] - t0;
  } else {
    t0 = st * state_len;
    S = state_len;
  }
  if (t0 < 0 || S < 1 || S > state_len || static_cast<long long>(t0) + S > T) {
    if (threadIdx.x == 0) report_status(BITRL_ERR_SHAPE, ATT_STAGE_BAD_STATE);
    return false;
  }
  return true;
}

__global__ void rope_table_kernel(float2* tab, int max_len, int hd, double theta) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  const int half = hd >> 1;
  if (idx >= max_len * half) return;
  const int p = idx / half, i = idx - p * half;
  const double ang = static_cast<double>(p) * pow(theta, -2.0 * static_cast<double>(i) / static_cast<double>(hd));
  tab[idx] = make_float2(static_cast<float>(cos(ang)), static_cast<float>(sin(ang)));
}

// The HD/32 consecutive elements a lane holds of one head row, rotated.  The partner of element e is e +- HD/2,
// which the lane 16 away holds at the same register index.
template <int HD>
__device__ __forceinline__ void rope_lane(const float (&x)[HD / 32], const float2* tab_row, int lane, float (&y)[HD / 32]) {
  constexpr int EPL = HD / 32;
#pragma unroll
  for (int j = 0; j < EPL; ++j) {
    const float partner = __shfl_xor_sync(0xffffffffu, x[j], 16);
    const int i = (lane * EPL + j) & (HD / 2 - 1);
    const float2 cs = tab_row[i];
    y[j] = fmaf(partner, lane < 16 ? -cs.y : cs.y, __fmul_rn(x[j], cs.x));
  }
}

template <int HD>
__device__ __forceinline__ void load_lane(const unsigned short* row, int lane, float (&x)[HD / 32]) {
  if constexpr (HD == 128) {
    const uint2 raw = *reinterpret_cast<const uint2*>(row + lane * 4);
    x[0] = __uint_as_float(raw.x << 16);
    x[1] = __uint_as_float(raw.x & 0xffff0000u);
    x[2] = __uint_as_float(raw.y << 16);
    x[3] = __uint_as_float(raw.y & 0xffff0000u);
  } else {
    const uint32_t raw = *reinterpret_cast<const uint32_t*>(row + lane * 2);
    x[0] = __uint_as_float(raw << 16);
    x[1] = __uint_as_float(raw & 0xffff0000u);
  }
}

// G = query heads of one kv head handled together (they share every key and value load); NCH = 32-key chunks.
template <int HD, int G, int NCH>
__global__ void __launch_bounds__(ATT_THREADS) attention_kernel(AttArgs a) {
  constexpr int EPL = HD / 32;   // elements of a head row per lane
  constexpr int KS = HD + 4;     // key row stride in floats: 16-byte rows, quarter-warps hit distinct banks
  constexpr int SMAX = NCH * 32;
  extern __shared__ __align__(16) float att_smem[];
  float* Ks = att_smem;                     // [SMAX][KS]   rotated keys
  float* Vs = Ks + SMAX * KS;               // [SMAX][HD]   values
  float* Qs = Vs + SMAX * HD;               // [warps][G][HD] rotated queries of the token a warp works on
  float* Ps = Qs + ATT_WARPS * G * HD;      // [warps][SMAX][G] unnormalized softmax weights

  pdl_enter();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int st = blockIdx.x / a.n_kv, kvh = blockIdx.x - st * a.n_kv;
  int t0, S;
  if (!state_range(a.state_off, a.state_len, a.T, st, t0, S)) return;
  if (S > SMAX) S = SMAX;  // the launcher picks NCH from state_len, so this never cuts
  const int rep = a.n_heads / a.n_kv;
  const int d = a.n_heads * HD, dkv = a.n_kv * HD, W = d + 2 * dkv;

  for (int r = warp; r < S; r += ATT_WARPS) {
    const unsigned short* krow = a.qkv + static_cast<long long>(t0 + r) * W + d + kvh * HD;
    float kx[EPL], ky[EPL], vx[EPL];
    load_lane<HD>(krow, lane, kx);
    load_lane<HD>(krow + dkv, lane, vx);
    rope_lane<HD>(kx, a.rope + r * (HD / 2), lane, ky);
#pragma unroll
    for (int j = 0; j < EPL; ++j) {
      Ks[r * KS + lane * EPL + j] = ky[j];
      Vs[r * HD + lane * EPL + j] = vx[j];
    }
  }
  __syncthreads();

  float* qw = Qs + warp * G * HD;
  float* pw = Ps + warp * SMAX * G;
  const float inv_sqrt = __fdiv_rn(1.0f, __fsqrt_rn(static_cast<float>(HD)));
  const int n_groups = rep / G;
  // Tokens are dealt to the warps in a zig-zag (w, 15-w, 16+w, 31-w, ...) so that every warp gets the same
  // number of causal keys.
  for (int k = 0; k * ATT_WARPS < S; ++k) {
    const int p = (k & 1) ? k * ATT_WARPS + (ATT_WARPS - 1 - warp) : k * ATT_WARPS + warp;
    if (p >= S) continue;
    const unsigned short* qrow = a.qkv + static_cast<long long>(t0 + p) * W;
    for (int grp = 0; grp < n_groups; ++grp) {
      const int h0 = kvh * rep + grp * G;
#pragma unroll
      for (int j = 0; j < G; ++j) {
        float qx[EPL], qy[EPL];
        load_lane<HD>(qrow + (h0 + j) * HD, lane, qx);
        rope_lane<HD>(qx, a.rope + p * (HD / 2), lane, qy);
#pragma unroll
        for (int e = 0; e < EPL; ++e) qw[j * HD + lane * EPL + e] = qy[e];
      }
      __syncwarp();

      // scores: lane = key r inside each 32-key chunk
      float sc[G][NCH];
#pragma unroll
      for (int c = 0; c < NCH; ++c) {
        const int r = c * 32 + lane;
        float acc[G];
#pragma unroll
        for (int j = 0; j < G; ++j) acc[j] = 0.0f;
        if (c * 32 <= p) {
          const float4* kr = reinterpret_cast<const float4*>(Ks + r * KS);
#pragma unroll 8
          for (int e4 = 0; e4 < HD / 4; ++e4) {
            const float4 kv = kr[e4];
#pragma unroll
            for (int j = 0; j < G; ++j) {
              const float4 qv = *reinterpret_cast<const float4*>(qw + j * HD + 4 * e4);
              acc[j] = fmaf(qv.x, kv.x, acc[j]);
              acc[j] = fmaf(qv.y, kv.y, acc[j]);
              acc[j] = fmaf(qv.z, kv.z, acc[j]);
              acc[j] = fmaf(qv.w, kv.w, acc[j]);
            }
          }
        }
#pragma unroll
        for (int j = 0; j < G; ++j) sc[j][c] = (r <= p) ? __fmul_rn(acc[j], inv_sqrt) : -INFINITY;
      }

      // softmax weights (unnormalized) and their sums
      float den[G];
#pragma unroll
      for (int j = 0; j < G; ++j) {
        float m = sc[j][0];
#pragma unroll
        for (int c = 1; c < NCH; ++c) m = fmaxf(m, sc[j][c]);
        m = warp_max(m);
        float s = 0.0f;
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
          const float w = (c * 32 + lane <= p) ? expf(sc[j][c] - m) : 0.0f;
          s += w;
          pw[(c * 32 + lane) * G + j] = w;
        }
        den[j] = warp_sum(s);
      }
      __syncwarp();

      // out = sum_r w_r v_r: lane = EPL consecutive elements of the head row
      float o[G][EPL];
#pragma unroll
      for (int j = 0; j < G; ++j)
#pragma unroll
        for (int e = 0; e < EPL; ++e) o[j][e] = 0.0f;
      for (int r = 0; r <= p; ++r) {
        float v[EPL], w[G];
#pragma unroll
        for (int e = 0; e < EPL; ++e) v[e] = Vs[r * HD + lane * EPL + e];
#pragma unroll
        for (int j = 0; j < G; ++j) w[j] = pw[r * G + j];
#pragma unroll
        for (int j = 0; j < G; ++j)
#pragma unroll
          for (int e = 0; e < EPL; ++e) o[j][e] = fmaf(w[j], v[e], o[j][e]);
      }
      unsigned short* orow = a.att + static_cast<long long>(t0 + p) * d;
#pragma unroll
      for (int j = 0; j < G; ++j) {
        uint32_t wd[EPL / 2];
#pragma unroll
        for (int e = 0; e < EPL; e += 2)
          wd[e / 2] = static_cast<uint32_t>(float_to_bf16_bits(__fdiv_rn(o[j][e], den[j]))) |
                      (static_cast<uint32_t>(float_to_bf16_bits(__fdiv_rn(o[j][e + 1], den[j]))) << 16);
        unsigned short* dst = orow + (h0 + j) * HD + lane * EPL;
        if constexpr (EPL == 4)
          *reinterpret_cast<uint2*>(dst) = make_uint2(wd[0], wd[1]);
        else
          *reinterpret_cast<uint32_t*>(dst) = wd[0];
      }
      __syncwarp();  // the next item overwrites this warp's query and weight rows
    }
  }
}

// ---- tensor-core formulation ------------------------------------------------------------------------------
// Same (state, kv head) decomposition, but scores and the weighted sum of values run on the warp-level tensor
// instruction mma.sync.m16n8k16 (f16 operands, fp32 accumulators).  To keep the products as exact as the fp32 form,
// every fp32 operand x is split into two halves x = hi + lo (hi = f16(x), lo = f16(x - hi): 22 significant bits) and
// the product a*b is formed as hi*hi + hi*lo + lo*hi (the dropped lo*lo term is below 2^-22 relative).  Values are
// bf16 numbers and convert to f16 exactly (down to 6e-5 in magnitude, 3e-8 absolute below); softmax weights are split.
// A warp owns one (query head, 16-token tile): Q fragments are read straight from global memory (the rotary partner
// of a dimension sits in the same lane four k-steps later), K/V fragments come from shared memory through ldmatrix.
constexpr int ATC_PAD = 8;  // halves added to each shared-memory row: consecutive rows start in different bank groups

__device__ __forceinline__ void mma_f16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// (x0, x1) -> f16x2 high parts and f16x2 low parts; x0 goes to the low half of the word.
__device__ __forceinline__ void split_f16x2(float x0, float x1, uint32_t& hi, uint32_t& lo) {
  const __half h0 = __float2half_rn(x0), h1 = __float2half_rn(x1);
  const __half l0 = __float2half_rn(x0 - __half2float(h0)), l1 = __float2half_rn(x1 - __half2float(h1));
  hi = static_cast<uint32_t>(__half_as_ushort(h0)) | (static_cast<uint32_t>(__half_as_ushort(h1)) << 16);
  lo = static_cast<uint32_t>(__half_as_ushort(l0)) | (static_cast<uint32_t>(__half_as_ushort(l1)) << 16);
}

// NKT = 8-key tiles held per query tile (keys padded to 8 * NKT, a multiple of 16).
template <int HD, int NKT>
__global__ void __launch_bounds__(ATT_THREADS) attention_tc_kernel(AttArgs a) {
  constexpr int KS = HD / 16;            // k-steps of the score product
  constexpr int ND = HD / 8;             // 8-wide output tiles
  constexpr int SP = NKT * 8;            // padded keys
  constexpr int RS = HD + ATC_PAD;       // shared-memory row stride in halves
  extern __shared__ __align__(16) unsigned char atc_smem[];
  __half* Khi = reinterpret_cast<__half*>(atc_smem);  // [SP][RS]
  __half* Klo = Khi + SP * RS;
  __half* Vh = Klo + SP * RS;

  pdl_enter();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int st = blockIdx.x / a.n_kv, kvh = blockIdx.x - st * a.n_kv;
  int t0, S;
  if (!state_range(a.state_off, a.state_len, a.T, st, t0, S)) return;
  if (S > SP) S = SP;  // the launcher picks NKT from state_len, so this never cuts
  const int rep = a.n_heads / a.n_kv;
  const int d = a.n_heads * HD, dkv = a.n_kv * HD, W = d + 2 * dkv;

  // ---- keys (rotated, split) and values of this state into shared memory; rows S..SP-1 are zero ----
  for (int r = warp; r < SP; r += ATT_WARPS) {
    __half* kh = Khi + r * RS;
    __half* kl = Klo + r * RS;
    __half* vh = Vh + r * RS;
    if (r < S) {
      const unsigned short* krow = a.qkv + static_cast<long long>(t0 + r) * W + d + kvh * HD;
      const float2* tab = a.rope + r * (HD / 2);
      for (int i = 2 * lane; i < HD / 2; i += 64) {  // dims i, i+1 and their partners i + HD/2, i + 1 + HD/2
        const uint32_t r1 = *reinterpret_cast<const uint32_t*>(krow + i);
        const uint32_t r2 = *reinterpret_cast<const uint32_t*>(krow + i + HD / 2);
        const float4 cs = *reinterpret_cast<const float4*>(tab + i);  // (cos_i, sin_i, cos_i+1, sin_i+1)
        const float x1a = __uint_as_float(r1 << 16), x1b = __uint_as_float(r1 & 0xffff0000u);
        const float x2a = __uint_as_float(r2 << 16), x2b = __uint_as_float(r2 & 0xffff0000u);
        uint32_t hi, lo;
        split_f16x2(fmaf(-x2a, cs.y, __fmul_rn(x1a, cs.x)), fmaf(-x2b, cs.w, __fmul_rn(x1b, cs.z)), hi, lo);
        *reinterpret_cast<uint32_t*>(kh + i) = hi;
        *reinterpret_cast<uint32_t*>(kl + i) = lo;
        split_f16x2(fmaf(x1a, cs.y, __fmul_rn(x2a, cs.x)), fmaf(x1b, cs.w, __fmul_rn(x2b, cs.z)), hi, lo);
        *reinterpret_cast<uint32_t*>(kh + i + HD / 2) = hi;
        *reinterpret_cast<uint32_t*>(kl + i + HD / 2) = lo;
      }
      for (int i = 2 * lane; i < HD; i += 64) {
        const uint32_t rv = *reinterpret_cast<const uint32_t*>(krow + dkv + i);
        const __half v0 = __float2half_rn(__uint_as_float(rv << 16)), v1 = __float2half_rn(__uint_as_float(rv & 0xffff0000u));
        *reinterpret_cast<uint32_t*>(vh + i) =
            static_cast<uint32_t>(__half_as_ushort(v0)) | (static_cast<uint32_t>(__half_as_ushort(v1)) << 16);
      }
    } else {
      for (int i = 2 * lane; i < HD; i += 64) {
        *reinterpret_cast<uint32_t*>(kh + i) = 0u;
        *reinterpret_cast<uint32_t*>(kl + i) = 0u;
        *reinterpret_cast<uint32_t*>(vh + i) = 0u;
      }
    }
  }
  __syncthreads();

  const int g = lane >> 2, t = lane & 3;
  const float inv_sqrt = __fdiv_rn(1.0f, __fsqrt_rn(static_cast<float>(HD)));
  const uint32_t khi_s = ptx_smem_u32(Khi), klo_s = ptx_smem_u32(Klo), vh_s = ptx_smem_u32(Vh);
  // ldmatrix row address of this lane: matrix lane/8, row lane%8
  const int lm = lane >> 3, lr = lane & 7;
  const int m_tiles = (S + 15) >> 4;
  for (int task = warp; task < rep * m_tiles; task += ATT_WARPS) {
    // larger query tiles first: they have more keys under the causal limit
    const int mt = m_tiles - 1 - task / rep, j = task % rep;
    const int head = kvh * rep + j;
    const int p_lo = 16 * mt + g, p_hi = p_lo + 8;
    const int nkt = min(NKT, 2 * mt + 2);  // key tiles under the causal limit of this query tile

    // ---- Q fragments: rows g and g+8 of the tile, rotated and split ----
    uint32_t qh[KS][4], ql[KS][4];
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      const int p = rr ? p_hi : p_lo;
      const bool live = p < S;
      const unsigned short* qrow = a.qkv + static_cast<long long>(t0 + (live ? p : 0)) * W + head * HD;
      const float2* tab = a.rope + (live ? p : 0) * (HD / 2);
#pragma unroll
      for (int ks = 0; ks < KS / 2; ++ks)
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          const int dim = 16 * ks + 8 * hf + 2 * t;  // dims dim, dim+1 (first half of the head) and their partners
          uint32_t r1 = 0u, r2 = 0u;
          if (live) {
            r1 = *reinterpret_cast<const uint32_t*>(qrow + dim);
            r2 = *reinterpret_cast<const uint32_t*>(qrow + dim + HD / 2);
          }
          const float4 cs = *reinterpret_cast<const float4*>(tab + dim);
          const float x1a = __uint_as_float(r1 << 16), x1b = __uint_as_float(r1 & 0xffff0000u);
          const float x2a = __uint_as_float(r2 << 16), x2b = __uint_as_float(r2 & 0xffff0000u);
          split_f16x2(fmaf(-x2a, cs.y, __fmul_rn(x1a, cs.x)), fmaf(-x2b, cs.w, __fmul_rn(x1b, cs.z)),
                      qh[ks][2 * hf + rr], ql[ks][2 * hf + rr]);
          split_f16x2(fmaf(x1a, cs.y, __fmul_rn(x2a, cs.x)), fmaf(x1b, cs.w, __fmul_rn(x2b, cs.z)),
                      qh[ks + KS / 2][2 * hf + rr], ql[ks + KS / 2][2 * hf + rr]);
        }
    }

    // ---- scores: c[nt] = Q K^T for key tile nt (rows g / g+8, keys 8nt+2t, +1) ----
    float c[NKT][4];
#pragma unroll
    for (int nt = 0; nt < NKT; ++nt) {
#pragma unroll
      for (int e = 0; e < 4; ++e) c[nt][e] = 0.0f;
      if (nt < nkt) {
#pragma unroll
        for (int ks = 0; ks < KS; ks += 2) {
          const uint32_t off = static_cast<uint32_t>(((8 * nt + lr) * RS + 16 * ks + 8 * lm) * 2);
          uint32_t bh[4], bl[4];
          ldmatrix_x4(khi_s + off, bh);
          ldmatrix_x4(klo_s + off, bl);
          mma_f16(c[nt], qh[ks], bh[0], bh[1]);
          mma_f16(c[nt], qh[ks], bl[0], bl[1]);
          mma_f16(c[nt], ql[ks], bh[0], bh[1]);
          mma_f16(c[nt], qh[ks + 1], bh[2], bh[3]);
          mma_f16(c[nt], qh[ks + 1], bl[2], bl[3]);
          mma_f16(c[nt], ql[ks + 1], bh[2], bh[3]);
        }
      }
    }

    // ---- softmax over the keys r <= p of each row (unnormalized weights, row sums kept) ----
    float m_lo = -INFINITY, m_hi = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < NKT; ++nt)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int key = 8 * nt + 2 * t + e;
        c[nt][e] = (nt < nkt && key <= p_lo) ? __fmul_rn(c[nt][e], inv_sqrt) : -INFINITY;
        c[nt][2 + e] = (nt < nkt && key <= p_hi) ? __fmul_rn(c[nt][2 + e], inv_sqrt) : -INFINITY;
        m_lo = fmaxf(m_lo, c[nt][e]);
        m_hi = fmaxf(m_hi, c[nt][2 + e]);
      }
    m_lo = fmaxf(m_lo, __shfl_xor_sync(0xffffffffu, m_lo, 1));
    m_lo = fmaxf(m_lo, __shfl_xor_sync(0xffffffffu, m_lo, 2));
    m_hi = fmaxf(m_hi, __shfl_xor_sync(0xffffffffu, m_hi, 1));
    m_hi = fmaxf(m_hi, __shfl_xor_sync(0xffffffffu, m_hi, 2));
    float s_lo = 0.0f, s_hi = 0.0f;
#pragma unroll
    for (int nt = 0; nt < NKT; ++nt)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        c[nt][e] = expf(c[nt][e] - m_lo);  // key 0 is never masked, so the maxima are finite
        c[nt][2 + e] = expf(c[nt][2 + e] - m_hi);
        s_lo += c[nt][e];
        s_hi += c[nt][2 + e];
      }
    s_lo += __shfl_xor_sync(0xffffffffu, s_lo, 1);
    s_lo += __shfl_xor_sync(0xffffffffu, s_lo, 2);
    s_hi += __shfl_xor_sync(0xffffffffu, s_hi, 1);
    s_hi += __shfl_xor_sync(0xffffffffu, s_hi, 2);

    // ---- out = P V: the score accumulators of two adjacent key tiles are the A fragment of one 16-key step ----
    float o[ND][4];
#pragma unroll
    for (int nd = 0; nd < ND; ++nd)
#pragma unroll
      for (int e = 0; e < 4; ++e) o[nd][e] = 0.0f;
#pragma unroll
    for (int kk = 0; kk < NKT / 2; ++kk) {
      if (2 * kk < nkt) {
        uint32_t ph[4], pl[4];
        split_f16x2(c[2 * kk][0], c[2 * kk][1], ph[0], pl[0]);
        split_f16x2(c[2 * kk][2], c[2 * kk][3], ph[1], pl[1]);
        split_f16x2(c[2 * kk + 1][0], c[2 * kk + 1][1], ph[2], pl[2]);
        split_f16x2(c[2 * kk + 1][2], c[2 * kk + 1][3], ph[3], pl[3]);
#pragma unroll
        for (int nd = 0; nd < ND; nd += 2) {
          uint32_t bv[4];
          ldmatrix_x4_trans(vh_s + static_cast<uint32_t>(((16 * kk + 8 * (lm & 1) + lr) * RS + 8 * (nd + (lm >> 1))) * 2), bv);
          mma_f16(o[nd], ph, bv[0], bv[1]);
          mma_f16(o[nd], pl, bv[0], bv[1]);
          mma_f16(o[nd + 1], ph, bv[2], bv[3]);
          mma_f16(o[nd + 1], pl, bv[2], bv[3]);
        }
      }
    }

    // ---- normalize, round to bf16, store rows g and g+8 ----
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      const int p = rr ? p_hi : p_lo;
      if (p < S) {
        const float den = rr ? s_hi : s_lo;
        unsigned short* orow = a.att + static_cast<long long>(t0 + p) * d + head * HD + 2 * t;
#pragma unroll
        for (int nd = 0; nd < ND; ++nd)
          *reinterpret_cast<uint32_t*>(orow + 8 * nd) =
              static_cast<uint32_t>(float_to_bf16_bits(__fdiv_rn(o[nd][2 * rr], den))) |
              (static_cast<uint32_t>(float_to_bf16_bits(__fdiv_rn(o[nd][2 * rr + 1], den))) << 16);
      }
    }
  }
}

template <int HD, int NKT>
bitrl_status launch_attention_tc_t(const AttArgs& a, int n_states, cudaStream_t st) {
  const size_t smem = static_cast<size_t>(3) * (NKT * 8) * (HD + ATC_PAD) * sizeof(__half);
  static bool attr_set[64] = {false};
  int dev = 0;
  BITRL_CUDA(cudaGetDevice(&dev));
  if (dev >= 0 && dev < 64 && !attr_set[dev]) {
    BITRL_CUDA(cudaFuncSetAttribute(attention_tc_kernel<HD, NKT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    static_cast<int>(smem)));
    attr_set[dev] = true;
  }
  BITRL_CUDA(launch_pdl(attention_tc_kernel<HD, NKT>, dim3(static_cast<unsigned>(n_states) * a.n_kv), dim3(ATT_THREADS),
                        smem, st, a));
  count_launch(1);
  return BITRL_OK;
}

template <int HD>
bitrl_status launch_attention_tc_hd(const AttArgs& a, int n_states, cudaStream_t st) {
  if (a.state_len <= 32) return launch_attention_tc_t<HD, 4>(a, n_states, st);
  if (a.state_len <= 64) return launch_attention_tc_t<HD, 8>(a, n_states, st);
  return launch_attention_tc_t<HD, 16>(a, n_states, st);
}

template <int HD, int G, int NCH>
bitrl_status launch_attention_t(const AttArgs& a, int n_states, cudaStream_t st) {
  constexpr int SMAX = NCH * 32;
  const size_t smem = sizeof(float) * (static_cast<size_t>(SMAX) * (HD + 4) + static_cast<size_t>(SMAX) * HD +
                                       static_cast<size_t>(ATT_WARPS) * G * HD + static_cast<size_t>(ATT_WARPS) * SMAX * G);
  static bool attr_set[64] = {false};
  int dev = 0;
  BITRL_CUDA(cudaGetDevice(&dev));
  if (dev >= 0 && dev < 64 && !attr_set[dev]) {
    BITRL_CUDA(cudaFuncSetAttribute(attention_kernel<HD, G, NCH>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    static_cast<int>(smem)));
    attr_set[dev] = true;
  }
  BITRL_CUDA(launch_pdl(attention_kernel<HD, G, NCH>, dim3(static_cast<unsigned>(n_states) * a.n_kv), dim3(ATT_THREADS),
                        smem, st, a));
  count_launch(1);
  return BITRL_OK;
}

template <int HD, int G>
bitrl_status launch_attention_g(const AttArgs& a, int n_states, cudaStream_t st) {
  if (a.state_len <= 32) return launch_attention_t<HD, G, 1>(a, n_states, st);
  if (a.state_len <= 64) return launch_attention_t<HD, G, 2>(a, n_states, st);
  return launch_attention_t<HD, G, 4>(a, n_states, st);
}

template <int HD>
bitrl_status launch_attention_hd(const AttArgs& a, int n_states, cudaStream_t st) {
  const int rep = a.n_heads / a.n_kv;
  if (rep % 4 == 0) return launch_attention_g<HD, 4>(a, n_states, st);
  if (rep % 2 == 0) return launch_attention_g<HD, 2>(a, n_states, st);
  return launch_attention_g<HD, 1>(a, n_states, st);
}

inline size_t rope_table_bytes(int max_state_len, int hd) {
  return (static_cast<size_t>(max_state_len) * (hd / 2) * sizeof(float2) + 255) / 256 * 256;
}

bitrl_status launch_rope_table(float2* tab, int max_state_len, int hd, double theta, cudaStream_t st) {
  const int n = max_state_len * (hd / 2);
  rope_table_kernel<<<(n + 255) / 256, 256, 0, st>>>(tab, max_state_len, hd, theta);
  count_launch(1);
  BITRL_CUDA(cudaGetLastError());
  return BITRL_OK;
}

// qkv -> att for all states; `rope` must hold the table of launch_rope_table for (state_len, hd, theta).
bitrl_status launch_attention(const void* qkv, int T, const int* state_off, int n_states, int state_len, int n_heads,
                              int n_kv, int hd, const float2* rope, void* att, cudaStream_t st) {
  AttArgs a{static_cast<const unsigned short*>(qkv), state_off, state_len, T, n_heads, n_kv, rope,
            static_cast<unsigned short*>(att)};
  if (hd == 128) return launch_attention_tc_hd<128>(a, n_states, st);
  if (hd == 64) return launch_attention_tc_hd<64>(a, n_states, st);
  return BITRL_ERR_SHAPE;
}

// Last-token pooling: out[s, :] = h[last token of state s, :]  (the latent h_t of Eq. 3, one per state).
__global__ void pool_last_token_kernel(const uint4* h, int T, const int* state_off, int state_len, int d8, uint4* out) {
  pdl_enter();
  const int st = blockIdx.x;
  int t0, S;
  if (!state_range(state_off, state_len, T, st, t0, S)) return;
  const uint4* src = h + static_cast<long long>(t0 + S - 1) * d8;
  uint4* dst = out + static_cast<long long>(st) * d8;
  for (int i = threadIdx.x; i < d8; i += blockDim.x) dst[i] = src[i];
}

bitrl_status launch_pool_last_token(const void* h, int T, const int* state_off, int n_states, int state_len, int d,
                                    void* out, cudaStream_t st) {
  BITRL_CUDA(launch_pdl(pool_last_token_kernel, dim3(n_states), dim3(128), 0, st, static_cast<const uint4*>(h), T,
                        state_off, state_len, d / 8, static_cast<uint4*>(out)));
  count_launch(1);
  return BITRL_OK;
}

}  // namespace bitrl
