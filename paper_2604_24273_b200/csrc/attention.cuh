// Attention inside each state of the frozen encoder (Eq. 3: h_t = f(serialize(s_t)); Sec. V: a state serializes
// to 15-40 tokens that go through the backbone in one forward pass).  Causal grouped-query attention with rotary
// position embedding, the form of the architecture the backbone follows (Sec. III-B cites it, the paper does not
// spell it out).  States are short and independent, so one CTA owns one (state, kv head): its rotated keys and its
// values sit in shared memory and every query tile of the heads that share the kv head runs over them.
//
//   rotary (rotate-half), position p = index of the token inside its state, i < head_dim/2:
//     angle = p * theta^(-2i/head_dim);  (x_i, x_{i+hd/2}) -> (x_i cos - x_{i+hd/2} sin, x_{i+hd/2} cos + x_i sin)
//   score(p, r) = q_p . k_r / sqrt(head_dim), r <= p;  w = exp(score - max);  out_p = (sum_r w_r v_r) / sum_r w_r
//
// The rotation is fp32 with cos/sin from an fp64 table rounded once; the two contractions run on the warp-level
// tensor instruction with split-precision operands (below); the output is rounded once to bf16.  Also here:
// last-token pooling of the encoder output to one latent per state.
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

// ---- the kernel ---------------------------------------------------------------------------------------------
// Scores and the weighted sum of values run on the warp-level tensor instruction mma.sync.m16n8k16 (f16 operands,
// fp32 accumulators; the contractions are 16..128 tokens wide, far below a tcgen05 tile).  To keep the products as
// exact as an fp32 multiply-add chain (which a first version of this kernel used: 76 us per block, bound by
// shared-memory wavefronts),
// every fp32 operand x is split into two halves x = hi + lo (hi = f16(x), lo = f16(x - hi): 22 significant bits) and
// the product a*b is formed as hi*hi + hi*lo + lo*hi (the dropped lo*lo term is below 2^-22 relative).  Values are
// bf16 numbers and convert to f16 exactly (down to 6e-5 in magnitude, 3e-8 absolute below); softmax weights are split.
// A warp owns one (query head, 16-token tile); all fragments come from shared memory through ldmatrix.
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

// Eight consecutive dimensions of the first half of a head row (x1) and their eight rotary partners (x2), rotated with
// cs = (cos, sin) of those eight dimensions, split, and stored as f16 high/low rows at columns c0 and c1.
__device__ __forceinline__ void rope_split_store8(const uint4& x1, const uint4& x2, const float4 (&cs)[4], __half* hi_row,
                                                  __half* lo_row, int c0, int c1) {
  const uint32_t w1[4] = {x1.x, x1.y, x1.z, x1.w}, w2[4] = {x2.x, x2.y, x2.z, x2.w};
  uint32_t h1[4], l1[4], h2[4], l2[4];
#pragma unroll
  for (int w = 0; w < 4; ++w) {
    const float x1a = __uint_as_float(w1[w] << 16), x1b = __uint_as_float(w1[w] & 0xffff0000u);
    const float x2a = __uint_as_float(w2[w] << 16), x2b = __uint_as_float(w2[w] & 0xffff0000u);
    split_f16x2(fmaf(-x2a, cs[w].y, __fmul_rn(x1a, cs[w].x)), fmaf(-x2b, cs[w].w, __fmul_rn(x1b, cs[w].z)), h1[w], l1[w]);
    split_f16x2(fmaf(x1a, cs[w].y, __fmul_rn(x2a, cs[w].x)), fmaf(x1b, cs[w].w, __fmul_rn(x2b, cs[w].z)), h2[w], l2[w]);
  }
  *reinterpret_cast<uint4*>(hi_row + c0) = make_uint4(h1[0], h1[1], h1[2], h1[3]);
  *reinterpret_cast<uint4*>(lo_row + c0) = make_uint4(l1[0], l1[1], l1[2], l1[3]);
  *reinterpret_cast<uint4*>(hi_row + c1) = make_uint4(h2[0], h2[1], h2[2], h2[3]);
  *reinterpret_cast<uint4*>(lo_row + c1) = make_uint4(l2[0], l2[1], l2[2], l2[3]);
}
// Eight bf16 values -> eight f16 values (exact for the magnitudes of activations).
__device__ __forceinline__ uint4 bf16x8_to_f16x8(const uint4& x) {
  const uint32_t w[4] = {x.x, x.y, x.z, x.w};
  uint32_t o[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const __half a = __float2half_rn(__uint_as_float(w[i] << 16)), b = __float2half_rn(__uint_as_float(w[i] & 0xffff0000u));
    o[i] = static_cast<uint32_t>(__half_as_ushort(a)) | (static_cast<uint32_t>(__half_as_ushort(b)) << 16);
  }
  return make_uint4(o[0], o[1], o[2], o[3]);
}

// NKT = 8-key tiles held per query tile (keys padded to 8 * NKT, a multiple of 16).
// STAGED: the rotated, split queries of all heads of the kv group are staged in shared memory by the same cooperative
// pass that stages keys and values (every global load of the CTA is a 16-byte load issued up front, one memory
// latency for the whole CTA); otherwise (long states or many heads per kv head, which would not fit) each warp builds
// the query fragments of its task from global memory.
template <int HD, int NKT, bool STAGED>
__global__ void __launch_bounds__(ATT_THREADS, NKT <= 4 ? 2 : 1) attention_tc_kernel(AttArgs a) {
  constexpr int KS = HD / 16;            // k-steps of the score product
  constexpr int ND = HD / 8;             // 8-wide output tiles
  constexpr int SP = NKT * 8;            // padded keys
  constexpr int RS = HD + ATC_PAD;       // shared-memory row stride in halves
  extern __shared__ __align__(16) unsigned char atc_smem[];
  __half* Khi = reinterpret_cast<__half*>(atc_smem);  // [SP][RS]
  __half* Klo = Khi + SP * RS;
  __half* Vh = Klo + SP * RS;
  __half* Qhi = Vh + SP * RS;  // STAGED: [rep * SP][RS], then Qlo the same

  pdl_enter();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int st = blockIdx.x / a.n_kv, kvh = blockIdx.x - st * a.n_kv;
  int t0, S;
  if (!state_range(a.state_off, a.state_len, a.T, st, t0, S)) return;
  if (S > SP) S = SP;  // the launcher picks NKT from state_len, so this never cuts
  const int rep = a.n_heads / a.n_kv;
  const int d = a.n_heads * HD, dkv = a.n_kv * HD, W = d + 2 * dkv;

  __half* Qlo = Qhi + rep * SP * RS;
  // ---- keys (rotated, split), values and (STAGED) queries of this state into shared memory; rows S..SP-1 are zero.
  // A thread owns eight dimensions of the first half of a row together with their eight rotary partners.
  {
    constexpr int CPR = HD / 16;  // such chunk pairs per row
    const int frow = threadIdx.x / CPR, cp = threadIdx.x % CPR;
    const int c0 = 8 * cp, c1 = HD / 2 + 8 * cp;
    for (int r = frow; r < SP; r += ATT_THREADS / CPR) {
      if (r < S) {
        const unsigned short* row = a.qkv + static_cast<long long>(t0 + r) * W;
        const unsigned short* krow = row + d + kvh * HD;
        const float4* tab = reinterpret_cast<const float4*>(a.rope + r * (HD / 2) + c0);
        const float4 cs[4] = {tab[0], tab[1], tab[2], tab[3]};
        const uint4 k1 = *reinterpret_cast<const uint4*>(krow + c0), k2 = *reinterpret_cast<const uint4*>(krow + c1);
        const uint4 v1 = *reinterpret_cast<const uint4*>(krow + dkv + c0), v2 = *reinterpret_cast<const uint4*>(krow + dkv + c1);
        if constexpr (STAGED) {
          for (int j0 = 0; j0 < rep; j0 += 4) {
            uint4 q1[4], q2[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
              if (j0 + i < rep) {
                const unsigned short* qrow = row + (kvh * rep + j0 + i) * HD;
                q1[i] = *reinterpret_cast<const uint4*>(qrow + c0);
                q2[i] = *reinterpret_cast<const uint4*>(qrow + c1);
              }
#pragma unroll
            for (int i = 0; i < 4; ++i)
              if (j0 + i < rep)
                rope_split_store8(q1[i], q2[i], cs, Qhi + ((j0 + i) * SP + r) * RS, Qlo + ((j0 + i) * SP + r) * RS, c0, c1);
          }
        }
        rope_split_store8(k1, k2, cs, Khi + r * RS, Klo + r * RS, c0, c1);
        *reinterpret_cast<uint4*>(Vh + r * RS + c0) = bf16x8_to_f16x8(v1);
        *reinterpret_cast<uint4*>(Vh + r * RS + c1) = bf16x8_to_f16x8(v2);
      } else {
        const uint4 z = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int c = h ? c1 : c0;
          *reinterpret_cast<uint4*>(Khi + r * RS + c) = z;
          *reinterpret_cast<uint4*>(Klo + r * RS + c) = z;
          *reinterpret_cast<uint4*>(Vh + r * RS + c) = z;
          if constexpr (STAGED)
            for (int j = 0; j < rep; ++j) {
              *reinterpret_cast<uint4*>(Qhi + (j * SP + r) * RS + c) = z;
              *reinterpret_cast<uint4*>(Qlo + (j * SP + r) * RS + c) = z;
            }
        }
      }
    }
  }
  __syncthreads();

  const int g = lane >> 2, t = lane & 3;
  const float inv_sqrt = __fdiv_rn(1.0f, __fsqrt_rn(static_cast<float>(HD)));
  const uint32_t khi_s = ptx_smem_u32(Khi), klo_s = ptx_smem_u32(Klo), vh_s = ptx_smem_u32(Vh);
  const uint32_t qhi_s = ptx_smem_u32(Qhi), qlo_s = ptx_smem_u32(Qlo);
  // ldmatrix row address of this lane: matrix lane/8, row lane%8
  const int lm = lane >> 3, lr = lane & 7;
  const int m_tiles = (S + 15) >> 4;
  for (int task = warp; task < rep * m_tiles; task += ATT_WARPS) {
    // larger query tiles first: they have more keys under the causal limit
    const int mt = m_tiles - 1 - task / rep, j = task % rep;
    const int head = kvh * rep + j;
    const int p_lo = 16 * mt + g, p_hi = p_lo + 8;
    const int nkt = min(NKT, 2 * mt + 2);  // key tiles under the causal limit of this query tile

    // ---- Q fragments of the tile (rows g and g+8 per lane), rotated and split ----
    uint32_t qh[STAGED ? 2 : KS][4], ql[STAGED ? 2 : KS][4];
    if constexpr (!STAGED) {
      // straight from global memory: the rotary partner of a dimension sits in the same lane KS/2 k-steps later
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
    }
    // STAGED: fragments come from shared memory, two k-steps at a time (matrix lm: rows 8 (lm & 1).., columns 8 (lm >> 1)..)
    const uint32_t q_off = static_cast<uint32_t>(((j * SP + 16 * mt + 8 * (lm & 1) + lr) * RS + 8 * (lm >> 1)) * 2);

    // ---- scores: c[nt] = Q K^T for key tile nt (rows g / g+8, keys 8nt+2t, +1) ----
    // Consecutive tensor instructions go to different accumulators (four key tiles, and the terms that involve a low
    // half are summed apart in c2), so that none waits for the one before it; the two sums are added at the end.
    float c[NKT][4], c2[NKT][4];
#pragma unroll
    for (int nt = 0; nt < NKT; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) c[nt][e] = c2[nt][e] = 0.0f;
#pragma unroll
    for (int n0 = 0; n0 < NKT; n0 += 4) {
      if (n0 < nkt) {
#pragma unroll
        for (int ks = 0; ks < KS; ks += 2) {
          const int k0 = STAGED ? 0 : ks, k1 = STAGED ? 1 : ks + 1;  // where this pair of k-steps sits in qh / ql
          if constexpr (STAGED) {
            ldmatrix_x4(qhi_s + q_off + 32 * ks, qh[0]);
            ldmatrix_x4(qlo_s + q_off + 32 * ks, ql[0]);
            ldmatrix_x4(qhi_s + q_off + 32 * ks + 32, qh[1]);
            ldmatrix_x4(qlo_s + q_off + 32 * ks + 32, ql[1]);
          }
          uint32_t bh[4][4], bl[4][4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            // key tiles beyond the causal limit hold finite numbers (keys of this state or zero rows) and are masked below
            const uint32_t off = static_cast<uint32_t>(((8 * (n0 + i) + lr) * RS + 16 * ks + 8 * lm) * 2);
            ldmatrix_x4(khi_s + off, bh[i]);
            ldmatrix_x4(klo_s + off, bl[i]);
          }
#pragma unroll
          for (int i = 0; i < 4; ++i) mma_f16(c[n0 + i], qh[k0], bh[i][0], bh[i][1]);
#pragma unroll
          for (int i = 0; i < 4; ++i) mma_f16(c2[n0 + i], qh[k0], bl[i][0], bl[i][1]);
#pragma unroll
          for (int i = 0; i < 4; ++i) mma_f16(c[n0 + i], qh[k1], bh[i][2], bh[i][3]);
#pragma unroll
          for (int i = 0; i < 4; ++i) mma_f16(c2[n0 + i], ql[k0], bh[i][0], bh[i][1]);
#pragma unroll
          for (int i = 0; i < 4; ++i) mma_f16(c2[n0 + i], qh[k1], bl[i][2], bl[i][3]);
#pragma unroll
          for (int i = 0; i < 4; ++i) mma_f16(c2[n0 + i], ql[k1], bh[i][2], bh[i][3]);
        }
      }
    }
#pragma unroll
    for (int nt = 0; nt < NKT; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) c[nt][e] += c2[nt][e];

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
        const float rden = __fdiv_rn(1.0f, rr ? s_hi : s_lo);  // one division per row, then multiplies
        unsigned short* orow = a.att + static_cast<long long>(t0 + p) * d + head * HD + 2 * t;
#pragma unroll
        for (int nd = 0; nd < ND; ++nd) {
          const __nv_bfloat162 pr = __floats2bfloat162_rn(__fmul_rn(o[nd][2 * rr], rden), __fmul_rn(o[nd][2 * rr + 1], rden));
          *reinterpret_cast<uint32_t*>(orow + 8 * nd) = *reinterpret_cast<const uint32_t*>(&pr);
        }
      }
    }
  }
}

template <int HD, int NKT, bool STAGED>
bitrl_status launch_attention_tc_t(const AttArgs& a, int n_states, cudaStream_t st) {
  const int rep = a.n_heads / a.n_kv;
  const size_t row_bytes = (HD + ATC_PAD) * sizeof(__half);
  const size_t smem = static_cast<size_t>(3 + (STAGED ? 2 * rep : 0)) * (NKT * 8) * row_bytes;
  static size_t attr_set[64] = {0};
  int dev = 0;
  BITRL_CUDA(cudaGetDevice(&dev));
  if (dev >= 0 && dev < 64 && attr_set[dev] < smem) {
    BITRL_CUDA(cudaFuncSetAttribute(attention_tc_kernel<HD, NKT, STAGED>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    static_cast<int>(smem)));
    attr_set[dev] = smem;
  }
  BITRL_CUDA(launch_pdl(attention_tc_kernel<HD, NKT, STAGED>, dim3(static_cast<unsigned>(n_states) * a.n_kv),
                        dim3(ATT_THREADS), smem, st, a));
  count_launch(1);
  return BITRL_OK;
}

template <int HD>
bitrl_status launch_attention_tc_hd(const AttArgs& a, int n_states, cudaStream_t st) {
  // queries are staged in shared memory while (3 + 2 * heads per kv head) * padded keys rows fit beside the rest
  const int rep = a.n_heads / a.n_kv;
  const auto fits = [&](int sp) { return static_cast<size_t>(3 + 2 * rep) * sp * (HD + ATC_PAD) * sizeof(__half) <= 200 * 1024; };
  if (a.state_len <= 32) return fits(32) ? launch_attention_tc_t<HD, 4, true>(a, n_states, st) : launch_attention_tc_t<HD, 4, false>(a, n_states, st);
  if (a.state_len <= 64) return fits(64) ? launch_attention_tc_t<HD, 8, true>(a, n_states, st) : launch_attention_tc_t<HD, 8, false>(a, n_states, st);
  return launch_attention_tc_t<HD, 16, false>(a, n_states, st);
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
