// a1+a2+a3 for M <= 16 tokens: the streaming (decode) kernel.  It is bound by the HBM stream of packed weights
// (N*K/4 bytes); activations are quantized in the prologue and the rescale is applied in the epilogue.
//
// Work split: one CTA of 8 warps owns 16 consecutive output rows.  The tile layout makes the 16 rows of one
// 128-wide k block a contiguous 512-byte piece: one 128-bit load per lane (lane = 2*row + half, 64 weights).
// Warp w takes k blocks w, w+8, ...  Codes are decoded four at a time with shift+mask into the byte lanes of
// a 32-bit word and multiplied with four int8 activations by one dp4a (codes are W_q+1, unsigned; the
// surplus sum_k x_q is subtracted once at the end).  Partial sums meet by one warp shuffle (the two k halves)
// and a shared-memory reduction over the 8 warps.
//
// Latency plan: a CTA's weights (up to 7 pieces per lane) are all requested before anything else, since they
// do not depend on the activations.  The kernel is launched with programmatic stream serialization: it signals
// its dependents at once and only waits for its predecessor (griddepcontrol.wait) after the weight loads are in
// flight, so the weight stream of launch i+1 overlaps the tail of launch i.  Every read of x / write of y comes
// after that wait.
#pragma once

#include "common.cuh"

namespace bitrl {

constexpr int GEMV_THREADS = 256;
constexpr int GEMV_WARPS = GEMV_THREADS / 32;
constexpr int GEMV_ROWS = 16;    // output rows per CTA
constexpr int GEMV_PREFETCH = 7;  // weight pieces per lane requested up front (covers K <= 7168)

struct GemvArgs {
  const uint8_t* tiles;
  const float* gamma;
  const unsigned short* x;  // bf16 bits [M,K] or null
  const int8_t* xq_in;      // [M,K] or null (then x is used)
  const float* absmax_in;   // [M] when xq_in is given
  int M, N, K;
  void* y;
  int out_dtype;
  const unsigned short* residual;
  int8_t* xq_out;
  float* absmax_out;
  int32_t* acc_out;
};

__device__ __forceinline__ float absmax8(const uint4& r) {
  const uint32_t w[4] = {r.x, r.y, r.z, r.w};
  float m = 0.0f;
#pragma unroll
  for (int i = 0; i < 4; ++i)
    m = fmaxf(m, fmaxf(fabsf(__uint_as_float(w[i] << 16)), fabsf(__uint_as_float(w[i] & 0xffff0000u))));
  return m;
}

template <int MT>
__device__ __forceinline__ void gemv_accumulate(const uint4& wv, const int8_t* xq_s, int K, int k0, int (&acc)[MT]) {
  const uint32_t wword[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const uint32_t c0 = wword[j] & 0x03030303u;
    const uint32_t c1 = (wword[j] >> 2) & 0x03030303u;
    const uint32_t c2 = (wword[j] >> 4) & 0x03030303u;
    const uint32_t c3 = (wword[j] >> 6) & 0x03030303u;
#pragma unroll
    for (int m = 0; m < MT; ++m) {
      const int4 xv = *reinterpret_cast<const int4*>(xq_s + m * K + k0 + 16 * j);
      acc[m] = dp4a_u8s8(c0, xv.x, acc[m]);
      acc[m] = dp4a_u8s8(c1, xv.y, acc[m]);
      acc[m] = dp4a_u8s8(c2, xv.z, acc[m]);
      acc[m] = dp4a_u8s8(c3, xv.w, acc[m]);
    }
  }
}

template <int MT>
__global__ void __launch_bounds__(GEMV_THREADS) gemv_kernel(GemvArgs a) {
  constexpr int WPR = MT >= GEMV_WARPS ? 1 : GEMV_WARPS / MT;  // warps that share one token row in the prologue
  constexpr int RPP = GEMV_WARPS / WPR;                        // token rows quantized per pass
  extern __shared__ __align__(16) unsigned char smem_raw[];
  int8_t* xq_s = reinterpret_cast<int8_t*>(smem_raw);  // [MT][K]
  __shared__ float redf[GEMV_WARPS];
  __shared__ int redi[GEMV_WARPS];
  __shared__ float scale_s[MT];
  __shared__ int rowsum_s[MT];
  __shared__ int part_s[GEMV_WARPS][GEMV_ROWS][MT];

  const int K = a.K, M = a.M;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int kblocks = K / TILE_K;
  const int groups = a.N / GEMV_ROWS;
  auto group_base = [&](int g) {
    return a.tiles + static_cast<size_t>(g >> 3) * kblocks * TILE_BYTES + (g & 7) * 512 + lane * 16;
  };

  // ---- weights of the first row group: they depend neither on the activations nor on the preceding kernel ----
  uint4 wreg[GEMV_PREFETCH];
  {
    const uint8_t* wb = group_base(blockIdx.x);
#pragma unroll
    for (int i = 0; i < GEMV_PREFETCH; ++i) {
      const int kb = warp + i * GEMV_WARPS;
      if (kb < kblocks) wreg[i] = __ldg(reinterpret_cast<const uint4*>(wb + static_cast<size_t>(kb) * TILE_BYTES));
    }
  }
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  // ---- prologue, once per CTA: quantized activations into shared memory (WPR warps per token row) ----
  const float gamma = *a.gamma;
  const int nvec8 = K >> 3;  // groups of 8 elements
  const int sub = warp % WPR;
#pragma unroll 1
  for (int pass = 0; pass < (MT + RPP - 1) / RPP; ++pass) {
    const int m = pass * RPP + warp / WPR;
    const bool live = m < M;
    uint2* dst = reinterpret_cast<uint2*>(xq_s + m * K);
    float amax = 1e-5f;
    int rs = 0;
    if (!live) {
      for (int i = sub * 32 + lane; i < nvec8; i += WPR * 32) dst[i] = make_uint2(0u, 0u);
    } else if (a.xq_in) {
      amax = a.absmax_in[m];
      const uint2* src = reinterpret_cast<const uint2*>(a.xq_in + static_cast<size_t>(m) * K);
      for (int i = sub * 32 + lane; i < nvec8; i += WPR * 32) {
        const uint2 wd = src[i];
        dst[i] = wd;
        rs = dp4a_u8s8(0x01010101u, static_cast<int>(wd.x), rs);
        rs = dp4a_u8s8(0x01010101u, static_cast<int>(wd.y), rs);
      }
    }
    const uint4* xr = reinterpret_cast<const uint4*>(a.x + static_cast<size_t>(live ? m : 0) * K);
    if (!a.xq_in) {  // uniform over the CTA: the block barriers below are reached by every thread
      float mx = 0.0f;
      if (live) {
#pragma unroll 4
        for (int i = sub * 32 + lane; i < nvec8; i += WPR * 32) mx = fmaxf(mx, absmax8(xr[i]));
      }
      mx = warp_max(mx);
      if (WPR > 1) {
        if (lane == 0) redf[warp] = mx;
        __syncthreads();
#pragma unroll
        for (int i = 0; i < WPR; ++i) mx = fmaxf(mx, redf[(warp / WPR) * WPR + i]);
      }
      amax = fmaxf(mx, 1e-5f);
      if (live) {
        const float inv = __fdiv_rn(127.0f, amax);
        uint2* xo = (a.xq_out && blockIdx.x == 0) ? reinterpret_cast<uint2*>(a.xq_out + static_cast<size_t>(m) * K) : nullptr;
#pragma unroll 2
        for (int i = sub * 32 + lane; i < nvec8; i += WPR * 32) {
          const uint4 raw = xr[i];
          const uint32_t rw[4] = {raw.x, raw.y, raw.z, raw.w};
          int q[8];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            q[2 * e] = quant_code(__uint_as_float(rw[e] << 16), inv);
            q[2 * e + 1] = quant_code(__uint_as_float(rw[e] & 0xffff0000u), inv);
          }
          uint2 wd;
          wd.x = (q[0] & 0xff) | ((q[1] & 0xff) << 8) | ((q[2] & 0xff) << 16) | (static_cast<uint32_t>(q[3]) << 24);
          wd.y = (q[4] & 0xff) | ((q[5] & 0xff) << 8) | ((q[6] & 0xff) << 16) | (static_cast<uint32_t>(q[7]) << 24);
          rs += q[0] + q[1] + q[2] + q[3] + q[4] + q[5] + q[6] + q[7];
          dst[i] = wd;
          if (xo) xo[i] = wd;
        }
      }
    }
    rs = warp_sum_i(rs);
    if (WPR > 1) {
      if (lane == 0) redi[warp] = rs;
      __syncthreads();
      rs = 0;
#pragma unroll
      for (int i = 0; i < WPR; ++i) rs += redi[(warp / WPR) * WPR + i];
    }
    if (sub == 0 && lane == 0 && m < MT) {
      rowsum_s[m] = live ? rs : 0;
      scale_s[m] = live ? out_scale(gamma, amax) : 0.0f;
      if (live && a.absmax_out && blockIdx.x == 0) a.absmax_out[m] = amax;
    }
  }
  __syncthreads();

  // ---- row groups of this CTA: weights of the next group are requested before the current one is consumed ----
  const int half = lane & 1;
  for (int g = blockIdx.x; g < groups; g += gridDim.x) {
    const uint8_t* wb = group_base(g);
    const int gn = g + gridDim.x;
    uint4 wnext[GEMV_PREFETCH];
    if (gn < groups) {
      const uint8_t* wbn = group_base(gn);
#pragma unroll
      for (int i = 0; i < GEMV_PREFETCH; ++i) {
        const int kb = warp + i * GEMV_WARPS;
        if (kb < kblocks) wnext[i] = __ldg(reinterpret_cast<const uint4*>(wbn + static_cast<size_t>(kb) * TILE_BYTES));
      }
    }
    int acc[MT];
#pragma unroll
    for (int m = 0; m < MT; ++m) acc[m] = 0;
#pragma unroll
    for (int i = 0; i < GEMV_PREFETCH; ++i) {
      const int kb = warp + i * GEMV_WARPS;
      if (kb < kblocks) gemv_accumulate<MT>(wreg[i], xq_s, K, kb * TILE_K + half * 64, acc);
    }
    for (int kb = warp + GEMV_PREFETCH * GEMV_WARPS; kb < kblocks; kb += GEMV_WARPS) {  // K > 7168 only
      const uint4 wv = __ldg(reinterpret_cast<const uint4*>(wb + static_cast<size_t>(kb) * TILE_BYTES));
      gemv_accumulate<MT>(wv, xq_s, K, kb * TILE_K + half * 64, acc);
    }

    // reduce: halves by shuffle, warps through shared memory
#pragma unroll
    for (int m = 0; m < MT; ++m) {
      acc[m] += __shfl_xor_sync(0xffffffffu, acc[m], 1);
      if (half == 0) part_s[warp][lane >> 1][m] = acc[m];
    }
    __syncthreads();

    // epilogue: one thread per (token, row)
    for (int idx = threadIdx.x; idx < GEMV_ROWS * MT; idx += GEMV_THREADS) {
      const int m = idx / GEMV_ROWS, r = idx % GEMV_ROWS;
      if (m >= M) continue;
      int t = 0;
#pragma unroll
      for (int w = 0; w < GEMV_WARPS; ++w) t += part_s[w][r][m];
      t -= rowsum_s[m];
      const size_t o = static_cast<size_t>(m) * a.N + static_cast<size_t>(g) * GEMV_ROWS + r;
      if (a.acc_out) a.acc_out[o] = t;
      const float yv = __fmul_rn(static_cast<float>(t), scale_s[m]);
      if (a.out_dtype == BITRL_OUT_F32) {
        static_cast<float*>(a.y)[o] = yv;
      } else {
        unsigned short yb = float_to_bf16_bits(yv);
        if (a.residual) yb = float_to_bf16_bits(__fadd_rn(bf16_bits_to_float(a.residual[o]), bf16_bits_to_float(yb)));
        static_cast<unsigned short*>(a.y)[o] = yb;
      }
    }
    if (gn < groups) {
      __syncthreads();  // part_s is reused by the next group
#pragma unroll
      for (int i = 0; i < GEMV_PREFETCH; ++i) wreg[i] = wnext[i];
    }
  }
}

int sm_count();

template <int MT>
bitrl_status launch_gemv_t(const GemvArgs& a, cudaStream_t st) {
  const size_t smem = static_cast<size_t>(MT) * a.K;
  if (smem > 32 * 1024)  // static arrays share the 48 KB default limit
    BITRL_CUDA(cudaFuncSetAttribute(gemv_kernel<MT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    static_cast<int>(smem)));
  cudaLaunchConfig_t cfg = {};
  const int groups = a.N / GEMV_ROWS, max_ctas = 2 * sm_count();  // persistent above two CTAs per SM
  cfg.gridDim = dim3(groups < max_ctas ? groups : max_ctas);
  cfg.blockDim = dim3(GEMV_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  BITRL_CUDA(cudaLaunchKernelEx(&cfg, gemv_kernel<MT>, a));
  count_launch(1);
  return BITRL_OK;
}

int gemv_q_max_m();

// Shared-memory budget of the streaming kernel: MT*K bytes of codes must fit beside the static arrays.
inline bool gemv_fits(int M, int K) {
  int mt = 1;
  while (mt < M) mt <<= 1;
  return M <= BITRL_GEMV_MAX_M && static_cast<size_t>(mt) * K <= 200 * 1024;
}

bitrl_status launch_gemv(const Linear* w, const void* x, const int8_t* xq, const float* absmax, int M, void* y,
                         int out_dtype, const void* residual, int8_t* xq_out, float* absmax_out,
                         int32_t* acc_out, cudaStream_t st) {
  GemvArgs a{w->tiles, w->gamma, static_cast<const unsigned short*>(x), xq, absmax, M, w->N, w->K, y, out_dtype,
             static_cast<const unsigned short*>(residual), xq_out, absmax_out, acc_out};
  if (M == 1) return launch_gemv_t<1>(a, st);
  if (M == 2) return launch_gemv_t<2>(a, st);
  if (M <= 4) return launch_gemv_t<4>(a, st);
  if (M <= 8) return launch_gemv_t<8>(a, st);
  return launch_gemv_t<16>(a, st);
}

}  // namespace bitrl
