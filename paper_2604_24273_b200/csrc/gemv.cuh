// a1+a2+a3 for M <= 16 tokens: the streaming (decode) kernel.  It is bound by the HBM stream of packed weights
// (N*K/4 bytes); activations are quantized in the prologue and the rescale is applied in the epilogue.
//
// Work split: one CTA of 8 warps owns 16 consecutive output rows.  The tile layout makes the 16 rows of one
// 128-wide k block a contiguous 512-byte piece: one 128-bit load per lane (lane = 2*row + half, 64 weights).
// Warp w takes k blocks w, w+8, ...  Codes are decoded four at a time with shift+mask into the byte lanes of
// a 32-bit word and multiplied with four int8 activations by one dp4a (codes are W_q+1, unsigned; the
// surplus sum_k x_q is subtracted once at the end).  Partial sums meet by one warp shuffle (the two k halves)
// and a shared-memory reduction over the 8 warps.
#pragma once

#include "common.cuh"

namespace bitrl {

constexpr int GEMV_THREADS = 256;
constexpr int GEMV_WARPS = GEMV_THREADS / 32;
constexpr int GEMV_ROWS = 16;  // output rows per CTA

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

template <int MT>
__global__ void __launch_bounds__(GEMV_THREADS) gemv_kernel(GemvArgs a) {
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
  const int row_tile = blockIdx.x >> 3, group = blockIdx.x & 7;
  const uint8_t* wbase = a.tiles + static_cast<size_t>(row_tile) * kblocks * TILE_BYTES + group * 512 + lane * 16;

  // The first weight piece does not depend on the activations: issue it before the prologue.
  uint4 wfirst = make_uint4(0x55555555u, 0x55555555u, 0x55555555u, 0x55555555u);
  if (warp < kblocks) wfirst = __ldg(reinterpret_cast<const uint4*>(wbase + static_cast<size_t>(warp) * TILE_BYTES));

  // ---- prologue: quantized activations into shared memory, per-token scale and row sum ----
  const float gamma = *a.gamma;
  const int nvec = K >> 2;
  for (int m = 0; m < MT; ++m) {
    if (m >= M) {
      for (int i = threadIdx.x; i < nvec; i += GEMV_THREADS) reinterpret_cast<uint32_t*>(xq_s + m * K)[i] = 0u;
      if (threadIdx.x == 0) { scale_s[m] = 0.0f; rowsum_s[m] = 0; }
      continue;
    }
    float amax;
    int rs = 0;
    if (a.xq_in) {
      amax = a.absmax_in[m];
      for (int i = threadIdx.x; i < nvec; i += GEMV_THREADS) {
        const uint32_t wd = reinterpret_cast<const uint32_t*>(a.xq_in + static_cast<size_t>(m) * K)[i];
        reinterpret_cast<uint32_t*>(xq_s + m * K)[i] = wd;
        rs = dp4a_u8s8(0x01010101u, static_cast<int>(wd), rs);
      }
    } else {
      const unsigned short* xr = a.x + static_cast<size_t>(m) * K;
      float mx = 0.0f;
      for (int i = threadIdx.x; i < nvec; i += GEMV_THREADS) {
        const uint2 raw = *reinterpret_cast<const uint2*>(xr + 4 * i);
        mx = fmaxf(mx, fmaxf(fmaxf(fabsf(__uint_as_float(raw.x << 16)), fabsf(__uint_as_float(raw.x & 0xffff0000u))),
                             fmaxf(fabsf(__uint_as_float(raw.y << 16)), fabsf(__uint_as_float(raw.y & 0xffff0000u)))));
      }
      mx = warp_max(mx);
      __syncthreads();
      if (lane == 0) redf[warp] = mx;
      __syncthreads();
      amax = 0.0f;
#pragma unroll
      for (int i = 0; i < GEMV_WARPS; ++i) amax = fmaxf(amax, redf[i]);
      amax = fmaxf(amax, 1e-5f);
      const float inv = __fdiv_rn(127.0f, amax);
      for (int i = threadIdx.x; i < nvec; i += GEMV_THREADS) {
        const uint2 raw = *reinterpret_cast<const uint2*>(xr + 4 * i);
        const int q0 = quant_code(__uint_as_float(raw.x << 16), inv);
        const int q1 = quant_code(__uint_as_float(raw.x & 0xffff0000u), inv);
        const int q2 = quant_code(__uint_as_float(raw.y << 16), inv);
        const int q3 = quant_code(__uint_as_float(raw.y & 0xffff0000u), inv);
        rs += q0 + q1 + q2 + q3;
        const uint32_t wd = (q0 & 0xff) | ((q1 & 0xff) << 8) | ((q2 & 0xff) << 16) | (static_cast<uint32_t>(q3) << 24);
        reinterpret_cast<uint32_t*>(xq_s + m * K)[i] = wd;
        if (a.xq_out && blockIdx.x == 0) reinterpret_cast<uint32_t*>(a.xq_out + static_cast<size_t>(m) * K)[i] = wd;
      }
    }
    rs = warp_sum_i(rs);
    __syncthreads();
    if (lane == 0) redi[warp] = rs;
    __syncthreads();
    if (threadIdx.x == 0) {
      int t = 0;
#pragma unroll
      for (int i = 0; i < GEMV_WARPS; ++i) t += redi[i];
      rowsum_s[m] = t;
      scale_s[m] = out_scale(gamma, amax);
      if (a.absmax_out && blockIdx.x == 0) a.absmax_out[m] = amax;
    }
  }
  __syncthreads();

  // ---- main loop: stream this warp's k blocks ----
  int acc[MT];
#pragma unroll
  for (int m = 0; m < MT; ++m) acc[m] = 0;
  const int half = lane & 1;
  uint4 wv = wfirst;
  for (int kb = warp; kb < kblocks; kb += GEMV_WARPS) {
    uint4 wnext = wv;
    if (kb + GEMV_WARPS < kblocks)
      wnext = __ldg(reinterpret_cast<const uint4*>(wbase + static_cast<size_t>(kb + GEMV_WARPS) * TILE_BYTES));
    const uint32_t wword[4] = {wv.x, wv.y, wv.z, wv.w};
    const int k0 = kb * TILE_K + half * 64;
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
    wv = wnext;
  }

  // ---- reduce: halves by shuffle, warps through shared memory ----
#pragma unroll
  for (int m = 0; m < MT; ++m) {
    acc[m] += __shfl_xor_sync(0xffffffffu, acc[m], 1);
    if (half == 0) part_s[warp][lane >> 1][m] = acc[m];
  }
  __syncthreads();

  // ---- epilogue: one thread per (token, row) ----
  for (int idx = threadIdx.x; idx < GEMV_ROWS * MT; idx += GEMV_THREADS) {
    const int m = idx / GEMV_ROWS, r = idx % GEMV_ROWS;
    if (m >= M) continue;
    int t = 0;
#pragma unroll
    for (int w = 0; w < GEMV_WARPS; ++w) t += part_s[w][r][m];
    t -= rowsum_s[m];
    const size_t o = static_cast<size_t>(m) * a.N + static_cast<size_t>(blockIdx.x) * GEMV_ROWS + r;
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
}

template <int MT>
bitrl_status launch_gemv_t(const GemvArgs& a, cudaStream_t st) {
  const size_t smem = static_cast<size_t>(MT) * a.K;
  if (smem > 32 * 1024)  // static arrays share the 48 KB default limit
    BITRL_CUDA(cudaFuncSetAttribute(gemv_kernel<MT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    static_cast<int>(smem)));
  gemv_kernel<MT><<<a.N / GEMV_ROWS, GEMV_THREADS, smem, st>>>(a);
  count_launch(1);
  BITRL_CUDA(cudaGetLastError());
  return BITRL_OK;
}

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
