// a1 and a4: per-token absmax int8 quantization, alone and fused behind the encoder's row producers
// (RMSNorm, V-repeat + RMSNorm, ReLU^2 gate + RMSNorm).  One CTA per token row; the row lives in shared memory
// as fp32 between the passes, so every activation tensor is read from HBM once and the codes written once.
#pragma once

#include "common.cuh"

namespace bitrl {

constexpr int ROW_THREADS = 256;

enum RowMode { ROW_PLAIN = 0, ROW_RMS = 1, ROW_VREPEAT = 2, ROW_RELU2 = 3 };

struct RowArgs {
  const unsigned short* in;  // bf16 bits
  long long in_stride;       // elements between consecutive rows of `in`
  int in_offset;             // first element of the row vector inside a row of `in`
  int gate_offset;           // ROW_RELU2: offset of `up` relative to g (= F)
  int Kv;                    // length of the row vector v that is normalized / quantized
  int rep;                   // ROW_VREPEAT: copies of each head; 1 otherwise
  int head_dim;              // ROW_VREPEAT: head width
  int Kout;                  // row length of xq / u_out (= Kv * rep)
  int8_t* xq;
  float* absmax;
  int32_t* rowsum;
  unsigned short* u_out;
};

__device__ __forceinline__ float block_sum(float v, float* red) {
  v = warp_sum(v);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = 0.0f;
#pragma unroll
  for (int i = 0; i < ROW_THREADS / 32; ++i) t += red[i];
  return t;
}
__device__ __forceinline__ float block_max(float v, float* red) {
  v = warp_max(v);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = 0.0f;
#pragma unroll
  for (int i = 0; i < ROW_THREADS / 32; ++i) t = fmaxf(t, red[i]);
  return t;
}
__device__ __forceinline__ int block_sum_i(int v, int* red) {
  v = warp_sum_i(v);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  int t = 0;
#pragma unroll
  for (int i = 0; i < ROW_THREADS / 32; ++i) t += red[i];
  return t;
}

template <int MODE>
__global__ void __launch_bounds__(ROW_THREADS) row_quant_kernel(RowArgs a) {
  extern __shared__ __align__(16) float vrow[];  // Kv floats
  __shared__ float redf[ROW_THREADS / 32];
  __shared__ int redi[ROW_THREADS / 32];

  const long long row = blockIdx.x;
  const unsigned short* src = a.in + row * a.in_stride + a.in_offset;
  const int nvec = a.Kv >> 2;  // groups of 4 elements (Kv is a multiple of 128)

  // pass 1: load, form v, keep it in shared memory, sum of squares in fp32
  float ss = 0.0f;
  for (int i = threadIdx.x; i < nvec; i += ROW_THREADS) {
    const uint2 raw = *reinterpret_cast<const uint2*>(src + 4 * i);
    float v0 = __uint_as_float(raw.x << 16), v1 = __uint_as_float(raw.x & 0xffff0000u);
    float v2 = __uint_as_float(raw.y << 16), v3 = __uint_as_float(raw.y & 0xffff0000u);
    if (MODE == ROW_RELU2) {
      const uint2 rawu = *reinterpret_cast<const uint2*>(src + a.gate_offset + 4 * i);
      const float u0 = __uint_as_float(rawu.x << 16), u1 = __uint_as_float(rawu.x & 0xffff0000u);
      const float u2 = __uint_as_float(rawu.y << 16), u3 = __uint_as_float(rawu.y & 0xffff0000u);
      v0 = fmaxf(v0, 0.0f); v1 = fmaxf(v1, 0.0f); v2 = fmaxf(v2, 0.0f); v3 = fmaxf(v3, 0.0f);
      v0 = __fmul_rn(__fmul_rn(v0, v0), u0);
      v1 = __fmul_rn(__fmul_rn(v1, v1), u1);
      v2 = __fmul_rn(__fmul_rn(v2, v2), u2);
      v3 = __fmul_rn(__fmul_rn(v3, v3), u3);
    }
    if (MODE != ROW_PLAIN) ss += v0 * v0 + v1 * v1 + v2 * v2 + v3 * v3;
    *reinterpret_cast<float4*>(vrow + 4 * i) = make_float4(v0, v1, v2, v3);
  }

  // pass 2: u = bf16(v * rstd); absmax of u
  float amax = 0.0f;
  if (MODE != ROW_PLAIN) {
    ss = block_sum(ss, redf);
    const float rstd = __fdiv_rn(1.0f, __fsqrt_rn(__fadd_rn(__fdiv_rn(ss, static_cast<float>(a.Kv)), 1e-5f)));
    for (int i = threadIdx.x; i < nvec; i += ROW_THREADS) {
      float4 v = *reinterpret_cast<float4*>(vrow + 4 * i);
      v.x = bf16_bits_to_float(float_to_bf16_bits(__fmul_rn(v.x, rstd)));
      v.y = bf16_bits_to_float(float_to_bf16_bits(__fmul_rn(v.y, rstd)));
      v.z = bf16_bits_to_float(float_to_bf16_bits(__fmul_rn(v.z, rstd)));
      v.w = bf16_bits_to_float(float_to_bf16_bits(__fmul_rn(v.w, rstd)));
      amax = fmaxf(amax, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
      *reinterpret_cast<float4*>(vrow + 4 * i) = v;
    }
  } else {
    for (int i = threadIdx.x; i < nvec; i += ROW_THREADS) {
      const float4 v = *reinterpret_cast<float4*>(vrow + 4 * i);
      amax = fmaxf(amax, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
    }
  }
  amax = fmaxf(block_max(amax, redf), 1e-5f);
  const float inv = __fdiv_rn(127.0f, amax);

  // pass 3: codes (and the optional bf16 copy of u), written `rep` times for the V-repeat producer
  int rs = 0;
  int8_t* xq = a.xq + row * a.Kout;
  unsigned short* uo = a.u_out ? a.u_out + row * a.Kout : nullptr;
  for (int i = threadIdx.x; i < nvec; i += ROW_THREADS) {
    const float4 v = *reinterpret_cast<float4*>(vrow + 4 * i);
    const int q0 = quant_code(v.x, inv), q1 = quant_code(v.y, inv), q2 = quant_code(v.z, inv),
              q3 = quant_code(v.w, inv);
    rs += q0 + q1 + q2 + q3;
    const uint32_t word = (q0 & 0xff) | ((q1 & 0xff) << 8) | ((q2 & 0xff) << 16) | (static_cast<uint32_t>(q3) << 24);
    uint2 ub;
    if (uo) {
      ub.x = static_cast<uint32_t>(float_to_bf16_bits(v.x)) | (static_cast<uint32_t>(float_to_bf16_bits(v.y)) << 16);
      ub.y = static_cast<uint32_t>(float_to_bf16_bits(v.z)) | (static_cast<uint32_t>(float_to_bf16_bits(v.w)) << 16);
    }
    if (MODE == ROW_VREPEAT) {
      const int k = 4 * i;
      const int kvh = k / a.head_dim, e = k - kvh * a.head_dim;
      for (int r = 0; r < a.rep; ++r) {
        const int ko = (kvh * a.rep + r) * a.head_dim + e;
        *reinterpret_cast<uint32_t*>(xq + ko) = word;
        if (uo) *reinterpret_cast<uint2*>(uo + ko) = ub;
      }
    } else {
      *reinterpret_cast<uint32_t*>(xq + 4 * i) = word;
      if (uo) *reinterpret_cast<uint2*>(uo + 4 * i) = ub;
    }
  }
  rs = block_sum_i(rs, redi);
  if (threadIdx.x == 0) {
    a.absmax[row] = amax;
    if (a.rowsum) a.rowsum[row] = rs * a.rep;
  }
}

// Register-resident variant: WPR warps share one row and every lane keeps its (up to) 7 groups of 8 values in
// registers across the three passes, so the row is read from global memory exactly once and no pass goes through
// shared memory; only the three scalar reductions cross warps.  8 / WPR rows per CTA.
constexpr int ROWQ_MAXG = 7;

// Four int32 codes -> four saturated int8 in one word (q0 in the low byte): two pack-with-saturation conversions.
__device__ __forceinline__ uint32_t pack_s8x4(int q0, int q1, int q2, int q3) {
  uint32_t hi, d;
  asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(q3), "r"(q2), "r"(0));
  asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(q1), "r"(q0), "r"(hi));
  return d;
}
// Sum of the four signed bytes of a word, added to acc.
__device__ __forceinline__ int dp4a_ones(uint32_t w, int acc) {
  int d;
  asm("dp4a.s32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(w), "r"(0x01010101), "r"(acc));
  return d;
}

template <int MODE, int WPR, int NG>
__global__ void __launch_bounds__(ROW_THREADS) row_quant_reg_kernel(RowArgs a, int T) {
  __shared__ float red_ss[ROW_THREADS / 32];
  __shared__ float red_mx[ROW_THREADS / 32];
  __shared__ int red_rs[ROW_THREADS / 32];
  pdl_enter();
  constexpr int ROWS = ROW_THREADS / 32 / WPR;           // rows a CTA works on at a time
  constexpr int NRAW = MODE == ROW_RELU2 ? 2 * NG : NG;  // 16-byte words a lane holds of one row
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int sub = warp % WPR, grp = warp / WPR;
  const int nvec8 = a.Kv >> 3;

  // Persistent CTAs: the raw words of the NEXT row are requested before the current row is processed, so that the
  // memory system stays busy during the arithmetic (a one-row-per-CTA version showed no overlap of the two).
  auto request = [&](long long row, uint4 (&raw)[NRAW]) {
    const unsigned short* src = a.in + row * a.in_stride + a.in_offset;
#pragma unroll
    for (int gi = 0; gi < NG; ++gi) {
      const int i = (gi * WPR + sub) * 32 + lane;
      if (row < T && i < nvec8) {
        raw[gi] = *reinterpret_cast<const uint4*>(src + 8 * i);
        if (MODE == ROW_RELU2) raw[NG + gi] = *reinterpret_cast<const uint4*>(src + a.gate_offset + 8 * i);
      }
    }
  };

  constexpr bool PREFETCH = MODE == ROW_RELU2 || MODE == ROW_PLAIN;  // see launch_row_reg
  uint4 raw[NRAW], nxt[PREFETCH ? NRAW : 1];
  long long row = static_cast<long long>(blockIdx.x) * ROWS + grp;
  const long long stride = static_cast<long long>(gridDim.x) * ROWS;
  if constexpr (PREFETCH) request(row, raw);
  // every group of the CTA runs the same number of iterations (the CTA-wide barriers below need that)
  for (long long base = static_cast<long long>(blockIdx.x) * ROWS; base < T; base += stride, row += stride) {
    const bool live = row < T;
    if constexpr (PREFETCH) request(row + stride, nxt);

    // pass 1: the row vector v, its sum of squares and its largest magnitude in one sweep
    float v[NG][8];
    float ss = 0.0f, mx = 0.0f;
#pragma unroll
    for (int gi = 0; gi < NG; ++gi) {
      const int i = (gi * WPR + sub) * 32 + lane;
      if (live && i < nvec8) {
        uint4 rg;
        if constexpr (PREFETCH) rg = raw[gi];
        else rg = *reinterpret_cast<const uint4*>(a.in + row * a.in_stride + a.in_offset + 8 * i);
        const uint32_t rw[4] = {rg.x, rg.y, rg.z, rg.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          v[gi][2 * e] = __uint_as_float(rw[e] << 16);
          v[gi][2 * e + 1] = __uint_as_float(rw[e] & 0xffff0000u);
        }
        if (MODE == ROW_RELU2) {
          const uint4 rawu = raw[MODE == ROW_RELU2 ? NG + gi : gi];  // the gate producer always prefetches
          const uint32_t ru[4] = {rawu.x, rawu.y, rawu.z, rawu.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float g0 = fmaxf(v[gi][2 * e], 0.0f), g1 = fmaxf(v[gi][2 * e + 1], 0.0f);
            v[gi][2 * e] = __fmul_rn(__fmul_rn(g0, g0), __uint_as_float(ru[e] << 16));
            v[gi][2 * e + 1] = __fmul_rn(__fmul_rn(g1, g1), __uint_as_float(ru[e] & 0xffff0000u));
          }
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          if (MODE != ROW_PLAIN) ss = fmaf(v[gi][e], v[gi][e], ss);
          mx = fmaxf(mx, fabsf(v[gi][e]));
        }
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) v[gi][e] = 0.0f;
      }
    }
    if (MODE != ROW_PLAIN) ss = warp_sum(ss);
    mx = warp_max(mx);
    if (WPR > 1) {
      if (lane == 0) { red_ss[warp] = ss; red_mx[warp] = mx; }
      __syncthreads();
      ss = 0.0f;
#pragma unroll
      for (int i = 0; i < WPR; ++i) { ss += red_ss[grp * WPR + i]; mx = fmaxf(mx, red_mx[grp * WPR + i]); }
    }
    // u = bf16(v * rstd) is monotonic in |v| (one rounded multiply, one rounding to bf16), so the largest |u| of the
    // row is the image of the largest |v|: no second reduction over the normalized values.
    float rstd = 1.0f, amax = mx;
    if (MODE != ROW_PLAIN) {
      rstd = __fdiv_rn(1.0f, __fsqrt_rn(__fadd_rn(__fdiv_rn(ss, static_cast<float>(a.Kv)), 1e-5f)));
      amax = bf16_bits_to_float(float_to_bf16_bits(__fmul_rn(mx, rstd)));
    }
    amax = fmaxf(amax, 1e-5f);
    const float inv = __fdiv_rn(127.0f, amax);

    // pass 2: normalize, round to bf16, quantize (round-to-nearest-even conversion, saturating pack), row sum of codes
    int rs = 0;
    int8_t* xq = a.xq + (live ? row : 0) * a.Kout;
    unsigned short* uo = a.u_out ? a.u_out + (live ? row : 0) * a.Kout : nullptr;
#pragma unroll
    for (int gi = 0; gi < NG; ++gi) {
      const int i = (gi * WPR + sub) * 32 + lane;
      if (live && i < nvec8) {
        uint32_t ub[4];
        int q[8];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float lo = v[gi][2 * e], hi = v[gi][2 * e + 1];
          if (MODE != ROW_PLAIN) {
            const __nv_bfloat162 pr = __floats2bfloat162_rn(__fmul_rn(lo, rstd), __fmul_rn(hi, rstd));
            ub[e] = *reinterpret_cast<const uint32_t*>(&pr);
            lo = __uint_as_float(ub[e] << 16);
            hi = __uint_as_float(ub[e] & 0xffff0000u);
          } else if (a.u_out) {
            ub[e] = (__float_as_uint(lo) >> 16) | (__float_as_uint(hi) & 0xffff0000u);
          }
          q[2 * e] = __float2int_rn(__fmul_rn(lo, inv));
          q[2 * e + 1] = __float2int_rn(__fmul_rn(hi, inv));
        }
        uint2 wd;
        wd.x = pack_s8x4(q[0], q[1], q[2], q[3]);
        wd.y = pack_s8x4(q[4], q[5], q[6], q[7]);
        rs = dp4a_ones(wd.y, dp4a_ones(wd.x, rs));
        const uint4 ub4 = make_uint4(ub[0], ub[1], ub[2], ub[3]);
        if (MODE == ROW_VREPEAT) {
          const int k = 8 * i;
          const int kvh = k / a.head_dim, e0 = k - kvh * a.head_dim;
          for (int r = 0; r < a.rep; ++r) {
            const int ko = (kvh * a.rep + r) * a.head_dim + e0;
            *reinterpret_cast<uint2*>(xq + ko) = wd;
            if (uo) *reinterpret_cast<uint4*>(uo + ko) = ub4;
          }
        } else {
          *reinterpret_cast<uint2*>(xq + 8 * i) = wd;
          if (uo) *reinterpret_cast<uint4*>(uo + 8 * i) = ub4;
        }
      }
    }
    rs = warp_sum_i(rs);
    if (WPR > 1) {
      if (lane == 0) red_rs[warp] = rs;
      __syncthreads();
      rs = 0;
#pragma unroll
      for (int i = 0; i < WPR; ++i) rs += red_rs[grp * WPR + i];
    }
    if (live && sub == 0 && lane == 0) {
      a.absmax[row] = amax;
      if (a.rowsum) a.rowsum[row] = rs * a.rep;
    }
    if constexpr (PREFETCH) {
#pragma unroll
      for (int i = 0; i < NRAW; ++i) raw[i] = nxt[i];
    }
  }
}

int sm_count();

template <int MODE, int WPR, int NG>
bitrl_status launch_row_reg(const RowArgs& a, int T, cudaStream_t st) {
  const int rows_per_cta = ROW_THREADS / 32 / WPR;
  const int row_groups = (T + rows_per_cta - 1) / rows_per_cta;
  // persistent: as many CTAs as are resident at once, each walking its rows with the next row's loads in flight
  static int per_sm = 0;
  if (per_sm == 0) {
    int n = 0;
    BITRL_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, row_quant_reg_kernel<MODE, WPR, NG>, ROW_THREADS, 0));
    per_sm = n > 0 ? n : 1;
  }
  // The gate producer reads 4 F bytes per row from a tensor larger than L2 and gains from the prefetch (37 -> 27 us at
  // T = 4096); the others read a row that the preceding GEMM left in L2 and run best with one row group per CTA.
  // The plain quantizer reads activations that come from outside the layer (HBM) and prefetches as well.
  int grid = (MODE == ROW_RELU2 || MODE == ROW_PLAIN) ? sm_count() * per_sm : row_groups;
  if (grid > row_groups) grid = row_groups;
  BITRL_CUDA(launch_pdl(row_quant_reg_kernel<MODE, WPR, NG>, dim3(grid), dim3(ROW_THREADS), 0, st, a, T));
  count_launch(1);
  return BITRL_OK;
}

template <int MODE>
bitrl_status launch_row(const RowArgs& a, int T, cudaStream_t st) {
  // Rows of up to 8 * 32 * 7 * 8 = 14336 values fit the register-resident kernel (head_dim a multiple of 8 keeps
  // the 8-value groups of the V-repeat producer inside one head).  Few values per lane (NG <= 3 or 4) keep the
  // register count low, so that several CTAs per SM overlap their load, compute and store phases.
  const int nvec8 = a.Kv >> 3;
  if (a.Kv % 8 == 0 && a.head_dim % 8 == 0) {
    if (nvec8 <= 32 * 3) return launch_row_reg<MODE, 1, 3>(a, T, st);
    if (nvec8 <= 64 * 3) return launch_row_reg<MODE, 2, 3>(a, T, st);
    if (nvec8 <= 128 * 3) return launch_row_reg<MODE, 4, 3>(a, T, st);
    if (nvec8 <= 256 * 3) return launch_row_reg<MODE, 8, 3>(a, T, st);
    if (nvec8 <= 256 * 4) return launch_row_reg<MODE, 8, 4>(a, T, st);
    if (nvec8 <= 256 * ROWQ_MAXG) return launch_row_reg<MODE, 8, ROWQ_MAXG>(a, T, st);
  }
  const size_t smem = static_cast<size_t>(a.Kv) * sizeof(float);
  if (smem > 40 * 1024) {
    BITRL_CUDA(cudaFuncSetAttribute(row_quant_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    static_cast<int>(smem)));
  }
  row_quant_kernel<MODE><<<T, ROW_THREADS, smem, st>>>(a);
  count_launch(1);
  BITRL_CUDA(cudaGetLastError());
  return BITRL_OK;
}

bitrl_status launch_quant_act(const void* x, int M, int K, int8_t* xq, float* absmax, int32_t* rowsum,
                              cudaStream_t st) {
  RowArgs a{static_cast<const unsigned short*>(x), K, 0, 0, K, 1, K, K, xq, absmax, rowsum, nullptr};
  return launch_row<ROW_PLAIN>(a, M, st);
}

bitrl_status launch_rmsnorm_quant(const void* h, int T, int K, int8_t* xq, float* absmax, int32_t* rowsum,
                                  void* u_out, cudaStream_t st) {
  RowArgs a{static_cast<const unsigned short*>(h), K, 0, 0, K, 1, K, K, xq, absmax, rowsum,
            static_cast<unsigned short*>(u_out)};
  return launch_row<ROW_RMS>(a, T, st);
}

bitrl_status launch_vrepeat_rmsnorm_quant(const void* qkv, int T, int n_heads, int n_kv, int hd, int8_t* xq,
                                          float* absmax, int32_t* rowsum, void* u_out, cudaStream_t st) {
  const int d = n_heads * hd, dkv = n_kv * hd;
  RowArgs a{static_cast<const unsigned short*>(qkv), d + 2 * dkv, d + dkv, 0, dkv, n_heads / n_kv, hd, d,
            xq, absmax, rowsum, static_cast<unsigned short*>(u_out)};
  return launch_row<ROW_VREPEAT>(a, T, st);
}

bitrl_status launch_relu2gate_rmsnorm_quant(const void* gu, int T, int F, int8_t* xq, float* absmax,
                                            int32_t* rowsum, void* u_out, cudaStream_t st) {
  RowArgs a{static_cast<const unsigned short*>(gu), 2LL * F, 0, F, F, 1, F, F, xq, absmax, rowsum,
            static_cast<unsigned short*>(u_out)};
  return launch_row<ROW_RELU2>(a, T, st);
}

}  // namespace bitrl
