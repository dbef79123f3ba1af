// W4A8 layer, the "INT4 critic" of the paper's ablations (Sec. V, Table IV; the paper names the precision only):
// int4 weights with one symmetric absmax scale per matrix, two biased codes (q + 8) per byte, even k in the low
// nibble.  The contraction is the int32 one of the other layers: acc = sum_k x_q (c - 8) = sum_k x_q c - 8 sum_k x_q,
// so the codes are fed as unsigned bytes and the row sum of the activations repays the bias once per output.
//   M <= 16: streaming dp4a kernel over the packed bytes (N*K/2 bytes from HBM).
//   M  > 16: the codes are expanded to int8 into the caller's workspace and the W8A8 tensor-core kernel runs on them
//            (a first version: the expansion is an extra pass over N*K bytes per call).
#pragma once

#include "common.cuh"
#include "gemm_w8.cuh"

namespace bitrl {

struct Gemv4Args {
  const uint8_t* packed;  // [N, K/2]
  const float* scale;
  const unsigned short* x;  // bf16 [M,K]
  int M, N, K;
  void* y;
  int out_dtype;
  int8_t* xq_out;  // debug taps (may be null)
  float* absmax_out;
  int32_t* acc_out;
};

// The activations are quantized once per CTA into shared memory with the even and the odd k of every group of eight
// in separate words, which is the order the two nibble planes of a weight word come out in.
template <int MT, int R>
__global__ void __launch_bounds__(GV8_THREADS) gemv_w4_kernel(Gemv4Args a) {
  extern __shared__ __align__(16) unsigned char gv4_smem[];
  int8_t* xq_s = reinterpret_cast<int8_t*>(gv4_smem);           // [MT][K]: per token an even-k plane and an odd-k plane of K/2 bytes
  float* sc_s = reinterpret_cast<float*>(gv4_smem + MT * a.K);  // [MT] a_m / 127
  int* rs_s = reinterpret_cast<int*>(sc_s + MT);                // [MT] sum_k x_q
  pdl_enter();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int K = a.K, nvec8 = K >> 3;
  for (int m = warp; m < MT; m += GV8_THREADS / 32) {
    uint2* dst = reinterpret_cast<uint2*>(xq_s + m * K);
    if (m >= a.M) {
      for (int i = lane; i < nvec8; i += 32) dst[i] = make_uint2(0u, 0u);
      if (lane == 0) { sc_s[m] = 0.0f; rs_s[m] = 0; }
      continue;
    }
    const uint4* xr = reinterpret_cast<const uint4*>(a.x + static_cast<size_t>(m) * K);
    float mx = 0.0f;
#pragma unroll 4
    for (int i = lane; i < nvec8; i += 32) mx = fmaxf(mx, absmax8(xr[i]));
    const float amax = fmaxf(warp_max(mx), 1e-5f);
    const float inv = __fdiv_rn(127.0f, amax);
    uint2* tap = (a.xq_out && blockIdx.x == 0) ? reinterpret_cast<uint2*>(a.xq_out + static_cast<size_t>(m) * K) : nullptr;
    int rs = 0;
    for (int i = lane; i < nvec8; i += 32) {
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
      if (tap) tap[i] = wd;
      // even k and odd k of every eight into two planes of K/2 bytes: the lanes of a warp then read consecutive 16-byte
      // pieces of either plane (side by side in one plane, every activation load was a two-way bank conflict)
      uint32_t* plane = reinterpret_cast<uint32_t*>(xq_s + m * K);
      plane[i] = __byte_perm(wd.x, wd.y, 0x6420);
      plane[(K >> 3) + i] = __byte_perm(wd.x, wd.y, 0x7531);
    }
    rs = warp_sum_i(rs);
    if (lane == 0) {
      sc_s[m] = __fdiv_rn(amax, 127.0f);
      rs_s[m] = rs;
      if (a.absmax_out && blockIdx.x == 0) a.absmax_out[m] = amax;
    }
  }
  __syncthreads();

  const float wscale = *a.scale;
  const int nvec16 = K >> 5;  // 16-byte pieces of a packed row (32 weights each)
  // R rows per warp at a time; the launcher takes fewer when the matrix has too few rows to give every SM a CTA.
  for (int n0 = (blockIdx.x * (GV8_THREADS / 32) + warp) * R; n0 < a.N; n0 += gridDim.x * (GV8_THREADS / 32) * R) {
    const uint4* wr = reinterpret_cast<const uint4*>(a.packed + static_cast<size_t>(n0) * (K >> 1));
    int acc[R][MT];
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int m = 0; m < MT; ++m) acc[r][m] = 0;
#pragma unroll 2
    for (int i = lane; i < nvec16; i += 32) {
      uint4 wv[R];
#pragma unroll
      for (int r = 0; r < R; ++r) wv[r] = wr[static_cast<size_t>(r) * nvec16 + i];
#pragma unroll
      for (int m = 0; m < MT; ++m) {
        // word p of the piece holds k = 32 i + 8 p .. + 7; its activations are word 4 i + p of the even-k and odd-k planes
        const uint4 xa = *reinterpret_cast<const uint4*>(xq_s + m * K + 16 * i);
        const uint4 xb = *reinterpret_cast<const uint4*>(xq_s + m * K + (K >> 1) + 16 * i);
        const uint32_t xe[4] = {xa.x, xa.y, xa.z, xa.w}, xo[4] = {xb.x, xb.y, xb.z, xb.w};
#pragma unroll
        for (int r = 0; r < R; ++r) {
          const uint32_t ww[4] = {wv[r].x, wv[r].y, wv[r].z, wv[r].w};
#pragma unroll
          for (int p = 0; p < 4; ++p) {
            acc[r][m] = dp4a_u8s8(ww[p] & 0x0f0f0f0fu, static_cast<int>(xe[p]), acc[r][m]);
            acc[r][m] = dp4a_u8s8((ww[p] >> 4) & 0x0f0f0f0fu, static_cast<int>(xo[p]), acc[r][m]);
          }
        }
      }
    }
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int m = 0; m < MT; ++m) acc[r][m] = warp_sum_i(acc[r][m]);
    if (lane == 0) {
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int m = 0; m < MT; ++m) {
          if (m < a.M) {
            const int tv = acc[r][m] - 8 * rs_s[m];
            const float yv = __fmul_rn(static_cast<float>(tv), __fmul_rn(wscale, sc_s[m]));
            const size_t o = static_cast<size_t>(m) * a.N + n0 + r;
            if (a.acc_out) a.acc_out[o] = tv;
            if (a.out_dtype == BITRL_OUT_F32) static_cast<float*>(a.y)[o] = yv;
            else static_cast<unsigned short*>(a.y)[o] = float_to_bf16_bits(yv);
          }
        }
    }
  }
}

template <int MT, int R>
bitrl_status launch_gemv_w4_tr(const Gemv4Args& a, cudaStream_t st) {
  const size_t smem = static_cast<size_t>(MT) * a.K + 2 * MT * sizeof(float) + 16;
  BITRL_CUDA(cudaFuncSetAttribute(gemv_w4_kernel<MT, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
  int grid = sm_count() * (smem <= 100 * 1024 ? 2 : 1);
  const int rows_per_cta = (GV8_THREADS / 32) * R;
  const int row_groups = (a.N + rows_per_cta - 1) / rows_per_cta;
  if (grid > row_groups) grid = row_groups;
  BITRL_CUDA(launch_pdl(gemv_w4_kernel<MT, R>, dim3(grid), dim3(GV8_THREADS), smem, st, a));
  count_launch(1);
  return BITRL_OK;
}

template <int MT>
bitrl_status launch_gemv_w4_t(const Gemv4Args& a, cudaStream_t st) {
  // as for the int8 streaming kernel: at one token, fewer rows per warp when four would leave SMs without a CTA
  constexpr int RMAX = MT <= 4 ? 4 : 2;
  if constexpr (MT == 1) {
    const int ctas_wanted = sm_count();
    if (a.N / ((GV8_THREADS / 32) * 4) >= ctas_wanted) return launch_gemv_w4_tr<MT, 4>(a, st);
    if (a.N / ((GV8_THREADS / 32) * 2) >= ctas_wanted) return launch_gemv_w4_tr<MT, 2>(a, st);
    return launch_gemv_w4_tr<MT, 1>(a, st);
  } else {
    return launch_gemv_w4_tr<MT, RMAX>(a, st);
  }
}

bitrl_status launch_gemv_w4(const uint8_t* packed, const float* scale, int N, int K, const void* x, int M, void* y,
                            int out_dtype, int8_t* xq_out, float* absmax_out, int32_t* acc_out, cudaStream_t st) {
  Gemv4Args a{packed, scale, static_cast<const unsigned short*>(x), M, N, K, y, out_dtype, xq_out, absmax_out, acc_out};
  if (M == 1) return launch_gemv_w4_t<1>(a, st);
  if (M == 2) return launch_gemv_w4_t<2>(a, st);
  if (M <= 4) return launch_gemv_w4_t<4>(a, st);
  if (M <= 8) return launch_gemv_w4_t<8>(a, st);
  return launch_gemv_w4_t<16>(a, st);
}

// Quantize + pack (after w8_absmax_kernel has left max|W| in amax_bits): 8 weights -> 4 bytes per thread step.
__global__ void w4_quantize_kernel(const float4* W, long long n8, const unsigned int* amax_bits, uint32_t* packed, float* scale) {
  const float a = fmaxf(__uint_as_float(*amax_bits), 1e-20f);
  const float inv = __fdiv_rn(7.0f, a);
  for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < n8;
       i += static_cast<long long>(gridDim.x) * blockDim.x) {
    const float4 v0 = W[2 * i], v1 = W[2 * i + 1];
    const float vals[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
    uint32_t word = 0;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      float q = rintf(__fmul_rn(vals[e], inv));
      q = fminf(fmaxf(q, -8.0f), 7.0f);
      word |= static_cast<uint32_t>(static_cast<int>(q) + 8) << (4 * e);  // k even in the low nibble of its byte
    }
    packed[i] = word;
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) *scale = __fdiv_rn(a, 7.0f);
}

bitrl_status launch_w4_quantize(const float* W, int N, int K, uint8_t* packed, float* scale2, cudaStream_t st) {
  const long long n = static_cast<long long>(N) * K;
  unsigned int* amax_bits = reinterpret_cast<unsigned int*>(scale2 + 1);
  BITRL_CUDA(cudaMemsetAsync(amax_bits, 0, 4, st));
  const int grid = sm_count() * 8;
  w8_absmax_kernel<<<grid, 256, 0, st>>>(reinterpret_cast<const float4*>(W), n / 4, amax_bits);
  w4_quantize_kernel<<<grid, 256, 0, st>>>(reinterpret_cast<const float4*>(W), n / 8, amax_bits,
                                           reinterpret_cast<uint32_t*>(packed), scale2);
  count_launch(2);
  BITRL_CUDA(cudaGetLastError());
  return BITRL_OK;
}

// Packed codes -> int8 values q = c - 8 (row-major [N,K]), 16 weights per thread step.
__global__ void w4_expand_kernel(const uint2* packed, long long n16, uint4* out) {
  pdl_enter();
  for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < n16;
       i += static_cast<long long>(gridDim.x) * blockDim.x) {
    const uint2 p = packed[i];
    const uint32_t w[2] = {p.x, p.y};
    uint32_t o[4];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const uint32_t lo = w[h] & 0x0f0f0f0fu, hi = (w[h] >> 4) & 0x0f0f0f0fu;  // even k | odd k of 8 consecutive weights
      // interleave back to k order and remove the bias: per-byte subtraction of 8 never borrows (codes are 0..15,
      // biased to 0x80.. first)
      const uint32_t k0123 = __byte_perm(lo, hi, 0x5140), k4567 = __byte_perm(lo, hi, 0x7362);
      o[2 * h] = __vsub4(k0123, 0x08080808u);
      o[2 * h + 1] = __vsub4(k4567, 0x08080808u);
    }
    out[i] = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

bitrl_status launch_w4_expand(const uint8_t* packed, int N, int K, int8_t* out, cudaStream_t st) {
  const long long n16 = static_cast<long long>(N) * K / 16;
  BITRL_CUDA(launch_pdl(w4_expand_kernel, dim3(sm_count() * 8), dim3(256), 0, st, reinterpret_cast<const uint2*>(packed), n16,
                        reinterpret_cast<uint4*>(out)));
  count_launch(1);
  return BITRL_OK;
}

}  // namespace bitrl
